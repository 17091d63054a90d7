"""Thin ctypes binding of ``libfdg.so`` (see ``include/fdg.h``): argument marshalling only.

Every step of the training iteration runs inside the library's CUDA kernels.  PyTorch appears
here only as the owner of device memory (its caching allocator backs ``fdg_allocator``) and as
a convenient way to hand device pointers in.  Importing this module without the compiled
library, or creating a context without an sm_100 device, fails loudly: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfdg.so")

STATUS = {0: "FDG_OK", 1: "FDG_ERR_INVALID_ARG", 2: "FDG_ERR_BAD_SPLIT", 3: "FDG_ERR_UNSUPPORTED",
          4: "FDG_ERR_ARCH", 5: "FDG_ERR_OOM", 6: "FDG_ERR_CUDA", 7: "FDG_ERR_TIMEOUT", 8: "FDG_ERR_STATE"}

EXPORTS = ["fdg_create", "fdg_grid_sms", "fdg_param_count", "fdg_param_layout", "fdg_set_params", "fdg_set_params_worker", "fdg_params_worker",
           "fdg_grads_worker", "fdg_consensus_error", "fdg_step", "fdg_step_host", "fdg_wait_ingest", "fdg_join", "fdg_params",
           "fdg_grads", "fdg_trace", "fdg_set_lr", "fdg_stats", "fdg_module_times", "fdg_profile", "fdg_profile_read",
           "fdg_bias_grad_static", "fdg_static_last_error",
           "fdg_last_error", "fdg_destroy"]


class FdgError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status


class fdg_layer(C.Structure):
    _fields_ = [("kind", C.c_int32), ("c_in", C.c_int32), ("c_out", C.c_int32), ("stride", C.c_int32), ("flags", C.c_int32)]


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class fdg_allocator(C.Structure):
    _fields_ = [("alloc", ALLOC_FN), ("free", FREE_FN), ("user", C.c_void_p)]


class fdg_kernel_stat(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_uint64), ("ms", C.c_double), ("flops", C.c_double), ("bytes", C.c_double)]


class fdg_param_tensor(C.Structure):
    _fields_ = [("layer", C.c_int32), ("module", C.c_int32), ("role", C.c_int32), ("ndim", C.c_int32),
                ("shape", C.c_int64 * 4), ("offset", C.c_uint64), ("count", C.c_uint64)]


PARAM_ROLES = ["W", "b", "gamma", "beta", "Wp", "gamma_p", "beta_p"]     # fdg_param_role


class fdg_options(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("in_h", C.c_int32), ("in_w", C.c_int32), ("in_c", C.c_int32),
                ("num_classes", C.c_int32), ("serial", C.c_int32), ("kernel_path", C.c_int32),
                ("worker_groups", C.c_int32), ("streams", C.POINTER(C.c_void_p)), ("mixing", C.POINTER(C.c_double)),
                ("grid_sms", C.c_int32)]


_lib = None


def lib():
    """Load libfdg.so (raises if it has not been built) and declare the C signatures."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2509_05679_b200.build` (needs nvcc)")
        L = C.CDLL(LIB_PATH)
        vp, fp = C.c_void_p, C.POINTER(C.c_float)
        L.fdg_create.restype = C.c_int
        L.fdg_create.argtypes = [C.POINTER(fdg_layer), C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.c_int32, C.c_int32,
                                 C.c_float, C.POINTER(fdg_options), C.POINTER(fdg_allocator), C.POINTER(vp)]
        L.fdg_grid_sms.restype = C.c_int
        L.fdg_grid_sms.argtypes = [vp, C.POINTER(C.c_int32)]
        L.fdg_param_count.restype = C.c_int
        L.fdg_param_count.argtypes = [vp, C.POINTER(C.c_size_t)]
        L.fdg_param_layout.restype = C.c_int
        L.fdg_param_layout.argtypes = [vp, C.POINTER(fdg_param_tensor), C.c_int32, C.POINTER(C.c_int32)]
        L.fdg_set_params.restype = C.c_int
        L.fdg_set_params.argtypes = [vp, fp, C.c_size_t]
        L.fdg_set_params_worker.restype = C.c_int
        L.fdg_set_params_worker.argtypes = [vp, C.c_int32, fp, C.c_size_t]
        for name in ("fdg_params_worker", "fdg_grads_worker"):
            getattr(L, name).restype = C.c_int
            getattr(L, name).argtypes = [vp, C.c_int32, fp, C.c_size_t, C.POINTER(C.c_size_t)]
        L.fdg_consensus_error.restype = C.c_int
        L.fdg_consensus_error.argtypes = [vp, C.POINTER(C.c_double)]
        for name in ("fdg_step", "fdg_step_host"):
            getattr(L, name).restype = C.c_int
            getattr(L, name).argtypes = [vp, vp, vp, fp]
        for name in ("fdg_params", "fdg_grads"):
            getattr(L, name).restype = C.c_int
            getattr(L, name).argtypes = [vp, fp, C.c_size_t, C.POINTER(C.c_size_t)]
        L.fdg_trace.restype = C.c_int
        L.fdg_trace.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.c_int32]
        L.fdg_set_lr.restype = C.c_int
        L.fdg_set_lr.argtypes = [vp, C.c_float]
        L.fdg_wait_ingest.restype = C.c_int
        L.fdg_wait_ingest.argtypes = [vp]
        L.fdg_join.restype = C.c_int
        L.fdg_join.argtypes = [vp, vp]
        L.fdg_stats.restype = C.c_int
        L.fdg_stats.argtypes = [vp, C.POINTER(C.c_size_t), C.POINTER(C.c_uint64)]
        L.fdg_module_times.restype = C.c_int
        L.fdg_module_times.argtypes = [vp, fp, C.c_int32]
        L.fdg_profile.restype = C.c_int
        L.fdg_profile.argtypes = [vp, C.c_int32]
        L.fdg_profile_read.restype = C.c_int
        L.fdg_profile_read.argtypes = [vp, C.POINTER(fdg_kernel_stat), C.c_int32, C.POINTER(C.c_int32)]
        L.fdg_bias_grad_static.restype = C.c_int
        L.fdg_bias_grad_static.argtypes = [vp, C.c_int32, C.c_int64, C.c_int32, vp, vp]
        L.fdg_static_last_error.restype = C.c_char_p
        L.fdg_static_last_error.argtypes = []
        L.fdg_last_error.restype = C.c_char_p
        L.fdg_last_error.argtypes = [vp]
        L.fdg_destroy.restype = None
        L.fdg_destroy.argtypes = [vp]
        _lib = L
    return _lib


class _TorchAllocator:
    """fdg_allocator backed by torch's caching allocator; keeps the tensors alive until freed."""

    def __init__(self, device):
        import torch
        self.live = {}
        self.device = device

        def _alloc(nbytes, _user):
            try:
                t = torch.empty(int(nbytes), dtype=torch.uint8, device=self.device)
            except Exception:      # out of memory: report NULL, the library turns it into FDG_ERR_OOM
                return None
            self.live[t.data_ptr()] = t
            return t.data_ptr()

        def _free(ptr, _user):
            self.live.pop(ptr, None)

        self._a, self._f = ALLOC_FN(_alloc), FREE_FN(_free)
        self.struct = fdg_allocator(self._a, self._f, None)


def _ptr(x):
    """Device or host address of a torch tensor / numpy array / int."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


class Context:
    """Owns one ``fdg_ctx``.  Method names mirror the C entry points."""

    def __init__(self, layers: Sequence[Sequence[int]], split_points: Sequence[int], n_workers: int,
                 per_worker_batch: int, lr: float, *, dtype: str = "bf16", in_shape=(32, 32, 3), num_classes: int = 10,
                 serial: bool = False, kernel_path: int = 0, device: int = 0, use_torch_allocator: bool = True,
                 streams: Optional[Sequence[int]] = None, worker_groups: int = 0, mixing=None, grid_sms: int = 0):
        import torch
        L = lib()
        if not torch.cuda.is_available():
            raise FdgError(4, "no CUDA device: this library has no CPU path")
        torch.cuda.set_device(device)
        self.K = len(split_points) + 1
        self.M = n_workers * per_worker_batch
        self.dtype = dtype
        self.in_shape = tuple(in_shape)
        arr = (fdg_layer * len(layers))(*[fdg_layer(*[int(v) for v in l]) for l in layers])
        sp = (C.c_int32 * max(1, len(split_points)))(*[int(s) for s in split_points])
        self._streams = None
        if streams is not None:          # K cudaStream_t handles owned by the caller
            assert len(streams) == self.K
            self._streams = (C.c_void_p * self.K)(*[C.c_void_p(int(h_)) for h_ in streams])
        self._mixing = None
        if mixing is not None:           # N x N weight matrix P (row-major doubles); the library copies it
            self._mixing = np.ascontiguousarray(mixing, dtype=np.float64)
            assert self._mixing.shape == (n_workers, n_workers)
        opt = fdg_options({"fp32": 0, "bf16": 1}[dtype], int(in_shape[0]), int(in_shape[1]), int(in_shape[2]),
                          int(num_classes), int(serial), int(kernel_path), int(worker_groups),
                          C.cast(self._streams, C.POINTER(C.c_void_p)) if self._streams is not None else None,
                          self._mixing.ctypes.data_as(C.POINTER(C.c_double)) if self._mixing is not None else None, int(grid_sms))
        self._alloc = _TorchAllocator(torch.device("cuda", device)) if use_torch_allocator else None
        h = C.c_void_p()
        st = L.fdg_create(arr, len(layers), sp, self.K, n_workers, per_worker_batch, float(lr), C.byref(opt),
                          C.byref(self._alloc.struct) if self._alloc else None, C.byref(h))
        if st != 0:
            raise FdgError(st, (L.fdg_last_error(None) or b"").decode())
        self.h = h
        n = C.c_size_t()
        self._ck(L.fdg_param_count(self.h, C.byref(n)))
        self.n_params = n.value
        g = C.c_int32()
        self._ck(L.fdg_grid_sms(self.h, C.byref(g)))
        self.grid_sms = g.value          # SMs the persistent kernels are sized for (fdg_options.grid_sms, resolved)

    def _ck(self, st):
        if st != 0:
            raise FdgError(st, (lib().fdg_last_error(self.h) or b"").decode())

    def close(self):
        if getattr(self, "h", None):
            lib().fdg_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def param_layout(self):
        """[(layer, module, role name, shape tuple, offset, count)] in canonical order (fdg_param_layout)."""
        n = C.c_int32()
        self._ck(lib().fdg_param_layout(self.h, None, 0, C.byref(n)))
        arr = (fdg_param_tensor * max(1, n.value))()
        self._ck(lib().fdg_param_layout(self.h, arr, n.value, C.byref(n)))
        return [(int(a.layer), int(a.module), PARAM_ROLES[a.role], tuple(int(v) for v in a.shape[:a.ndim]), int(a.offset), int(a.count))
                for a in arr[:n.value]]

    def set_params(self, params: np.ndarray):
        p = np.ascontiguousarray(params, dtype=np.float32)
        self._ck(lib().fdg_set_params(self.h, p.ctypes.data_as(C.POINTER(C.c_float)), p.size))

    def set_params_worker(self, worker: int, params: np.ndarray):
        p = np.ascontiguousarray(params, dtype=np.float32)
        self._ck(lib().fdg_set_params_worker(self.h, int(worker), p.ctypes.data_as(C.POINTER(C.c_float)), p.size))

    def _vec_worker(self, fn, worker: int) -> np.ndarray:
        out = np.empty(self.n_params, dtype=np.float32)
        n = C.c_size_t()
        self._ck(fn(self.h, int(worker), out.ctypes.data_as(C.POINTER(C.c_float)), out.size, C.byref(n)))
        return out

    def params_worker(self, worker: int) -> np.ndarray:
        return self._vec_worker(lib().fdg_params_worker, worker)

    def grads_worker(self, worker: int) -> np.ndarray:
        return self._vec_worker(lib().fdg_grads_worker, worker)

    def consensus_error(self) -> float:
        d = C.c_double()
        self._ck(lib().fdg_consensus_error(self.h, C.byref(d)))
        return d.value

    def step(self, dev_inputs, dev_labels, want_loss: bool = False) -> Optional[float]:
        loss = C.c_float()
        self._ck(lib().fdg_step(self.h, _ptr(dev_inputs), _ptr(dev_labels), C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def step_host(self, host_inputs, host_labels, want_loss: bool = False) -> Optional[float]:
        loss = C.c_float()
        self._ck(lib().fdg_step_host(self.h, _ptr(host_inputs), _ptr(host_labels), C.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    def wait_ingest(self):
        self._ck(lib().fdg_wait_ingest(self.h))

    def join(self, stream: int = 0):
        """Make the caller's stream (a cudaStream_t handle) wait for all work enqueued so far."""
        self._ck(lib().fdg_join(self.h, stream or None))

    def _vec(self, fn) -> np.ndarray:
        out = np.empty(self.n_params, dtype=np.float32)
        n = C.c_size_t()
        self._ck(fn(self.h, out.ctypes.data_as(C.POINTER(C.c_float)), out.size, C.byref(n)))
        return out

    def params(self) -> np.ndarray:
        return self._vec(lib().fdg_params)

    def grads(self) -> np.ndarray:
        return self._vec(lib().fdg_grads)

    def trace(self):
        f, b, v = (np.empty(self.K, dtype=np.int64) for _ in range(3))
        p = lambda a: a.ctypes.data_as(C.POINTER(C.c_int64))
        self._ck(lib().fdg_trace(self.h, p(f), p(b), p(v), self.K))
        return f, b, v

    def set_lr(self, lr: float):
        self._ck(lib().fdg_set_lr(self.h, float(lr)))

    def stats(self):
        nb, nl = C.c_size_t(), C.c_uint64()
        self._ck(lib().fdg_stats(self.h, C.byref(nb), C.byref(nl)))
        return nb.value, nl.value

    def profile(self, enable: bool):
        self._ck(lib().fdg_profile(self.h, int(enable)))

    def profile_read(self):
        """{kernel class: dict(launches, ms, flops, bytes)} since profile(True)."""
        arr = (fdg_kernel_stat * 256)()
        n = C.c_int32()
        self._ck(lib().fdg_profile_read(self.h, arr, 256, C.byref(n)))
        return {arr[i].name.decode(): dict(launches=int(arr[i].launches), ms=arr[i].ms, flops=arr[i].flops, bytes=arr[i].bytes)
                for i in range(n.value)}

    def module_times(self) -> np.ndarray:
        ms = np.empty(self.K, dtype=np.float32)
        self._ck(lib().fdg_module_times(self.h, ms.ctypes.data_as(C.POINTER(C.c_float)), self.K))
        return ms


def bias_grad_static(dev_dy, dtype: str, rows: int, channels: int, dev_db, stream: int = 0) -> None:
    """dev_db[c] = sum_rows dev_dy[row][c] through fdg_bias_grad_static: no device memory is allocated
    by the call (its scratch is a fixed array inside the library).  Arguments are device tensors /
    addresses owned by the caller; raises FdgError with the library's message on a rejected call."""
    st = lib().fdg_bias_grad_static(_ptr(dev_dy), {"fp32": 0, "bf16": 1}[dtype], int(rows), int(channels), _ptr(dev_db), stream or None)
    if st != 0:
        raise FdgError(st, (lib().fdg_static_last_error() or b"").decode())


def to_device(net_dtype: str, x: np.ndarray):
    """Copy a host fp32 batch to the device in the context's storage dtype (plumbing for callers)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    t = t.to(torch.bfloat16).contiguous() if net_dtype == "bf16" else t
    torch.cuda.current_stream().synchronize()      # the library's streams do not wait for torch's
    return t
