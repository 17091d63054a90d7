"""ctypes front end of the CPU oracle (test infrastructure only; the product never imports it).

``build()`` compiles ``fdg_oracle.cpp`` with g++ into ``libfdg_oracle.so`` next to this file.
Everything numeric happens inside the C++ code; this file only marshals arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fdg_oracle.cpp")
_LIB = os.path.join(_HERE, "libfdg_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ftree-vectorize", "-fPIC", "-shared",
                               "-pthread", "-o", _LIB, _SRC])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        dp, ip, lp = C.POINTER(C.c_double), C.POINTER(C.c_int32), C.POINTER(C.c_int64)
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [ip, C.c_int, ip, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.c_int, dp, C.c_double]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_set_threads.argtypes = [C.c_int]
        L.orc_threads.restype = C.c_int
        L.orc_kink_margin.restype = C.c_double
        L.orc_kink_margin.argtypes = [C.c_int]
        L.orc_param_count.restype = C.c_size_t
        L.orc_param_count.argtypes = [C.c_void_p]
        L.orc_set_flag_use_current_weights.argtypes = [C.c_void_p, C.c_int]
        L.orc_set_storage_bf16.argtypes = [C.c_void_p, C.c_int]
        L.orc_round_bf16.argtypes = [dp, dp, C.c_size_t]
        L.orc_set_params.argtypes = [C.c_void_p, C.c_int, dp]
        L.orc_get_params.argtypes = [C.c_void_p, C.c_int, dp]
        L.orc_get_grads.argtypes = [C.c_void_p, C.c_int, dp]
        L.orc_trace.argtypes = [C.c_void_p, lp, lp, lp, lp]
        L.orc_step.restype = C.c_int
        L.orc_step.argtypes = [C.c_void_p, dp, ip, C.c_double, dp, lp]
        L.orc_plain_loss_grad.restype = C.c_double
        L.orc_plain_loss_grad.argtypes = [ip, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                          dp, dp, ip, C.c_double, dp]
        L.orc_plain_logits.argtypes = [ip, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, dp, dp, dp]
        L.orc_softmax_ce.restype = C.c_double
        L.orc_softmax_ce.argtypes = [dp, ip, C.c_int, C.c_int, C.c_double, dp]
        _lib = L
    return _lib


def _d(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _i(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _layers(layers) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(layers, dtype=np.int32).reshape(-1, 5))


def threads() -> int:
    return int(lib().orc_threads())


def kink_margin(reset: bool = True) -> float:
    """Smallest |x| at a ReLU / top-2 gap in a max-pool window since the last reset."""
    return float(lib().orc_kink_margin(int(reset)))


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


class Oracle:
    """All S*K agents of the method, simulated in one process in fp64."""

    def __init__(self, layers, splits, n_workers, batch, in_shape, classes, P=None, grad_scale=None):
        self.layers = _layers(layers)
        self.splits = np.asarray(list(splits), dtype=np.int32)
        self.K = len(self.splits) + 1
        self.S, self.B = int(n_workers), int(batch)
        self.in_shape = tuple(int(v) for v in in_shape)
        self.classes = int(classes)
        if grad_scale is None:
            grad_scale = 1.0 / self.B
        Pp = None
        if P is not None:
            self._P = np.ascontiguousarray(P, dtype=np.float64)
            assert self._P.shape == (self.S, self.S)
            Pp = _d(self._P)
        self.h = lib().orc_create(_i(self.layers), len(self.layers), _i(self.splits) if self.K > 1 else None,
                                  self.K, self.S, self.B, *self.in_shape, self.classes, Pp, float(grad_scale))
        if not self.h:
            raise ValueError("oracle rejected the split points")
        self.n_params = int(lib().orc_param_count(self.h))

    def __del__(self):
        if getattr(self, "h", None) and lib is not None:
            lib().orc_destroy(self.h)
            self.h = None

    def set_params(self, p, worker: int = -1):
        p = np.ascontiguousarray(p, dtype=np.float64)
        assert p.size == self.n_params
        lib().orc_set_params(self.h, worker, _d(p))

    def params(self, worker: int = 0) -> np.ndarray:
        out = np.empty(self.n_params, dtype=np.float64)
        lib().orc_get_params(self.h, worker, _d(out))
        return out

    def grads(self, worker: int = 0) -> np.ndarray:
        out = np.empty(self.n_params, dtype=np.float64)
        lib().orc_get_grads(self.h, worker, _d(out))
        return out

    def use_current_weights(self, on: bool):
        lib().orc_set_flag_use_current_weights(self.h, int(on))

    def storage_bf16(self, on: bool):
        """Round every tensor the bf16 configurations store in bf16 (see the C++ header comment)."""
        lib().orc_set_storage_bf16(self.h, int(on))

    def step(self, inputs, labels, lr):
        x = np.ascontiguousarray(inputs, dtype=np.float64)
        y = np.ascontiguousarray(labels, dtype=np.int32)
        assert x.size == self.S * self.B * int(np.prod(self.in_shape)) and y.size == self.S * self.B
        loss = C.c_double()
        lb = C.c_int64()
        lib().orc_step(self.h, _d(x), _i(y), float(lr), C.byref(loss), C.byref(lb))
        return loss.value, lb.value

    def trace(self):
        f, b, v, m = (np.empty(self.K, dtype=np.int64) for _ in range(4))
        p = lambda a: a.ctypes.data_as(C.POINTER(C.c_int64))
        lib().orc_trace(self.h, p(f), p(b), p(v), p(m))
        return f, b, v, m


def plain_loss_grad(layers, n_workers, batch, in_shape, params, inputs, labels, grad_scale=None, want_grad=True):
    L = _layers(layers)
    p = np.ascontiguousarray(params, dtype=np.float64)
    x = np.ascontiguousarray(inputs, dtype=np.float64)
    y = np.ascontiguousarray(labels, dtype=np.int32)
    if grad_scale is None:
        grad_scale = 1.0 / batch
    g = np.zeros_like(p) if want_grad else None
    loss = lib().orc_plain_loss_grad(_i(L), len(L), n_workers, batch, *in_shape, _d(p), _d(x), _i(y),
                                     float(grad_scale), _d(g) if want_grad else None)
    return float(loss), g


def plain_logits(layers, n_workers, batch, in_shape, params, inputs, classes):
    L = _layers(layers)
    p = np.ascontiguousarray(params, dtype=np.float64)
    x = np.ascontiguousarray(inputs, dtype=np.float64)
    out = np.empty((n_workers * batch, classes), dtype=np.float64)
    lib().orc_plain_logits(_i(L), len(L), n_workers, batch, *in_shape, _d(p), _d(x), _d(out))
    return out


def round_bf16(x) -> np.ndarray:
    a = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty_like(a)
    lib().orc_round_bf16(_d(a), _d(out), a.size)
    return out


def softmax_ce(logits, labels, scale=1.0):
    z = np.ascontiguousarray(logits, dtype=np.float64)
    y = np.ascontiguousarray(labels, dtype=np.int32)
    g = np.empty_like(z)
    loss = lib().orc_softmax_ce(_d(z), _i(y), z.shape[0], z.shape[1], float(scale), _d(g))
    return float(loss), g
