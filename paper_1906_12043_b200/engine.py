"""Thin ctypes binding over libcocod.so (the C boundary of include/cocod.h).

Argument marshalling only: every step of Algorithm 1's parameter path (local step, stored
copy, mean, merge) runs in the library's CUDA kernels.  torch is used for device memory and
streams.  There is no CPU fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcocod.so")

OK, ERR_INVALID, ERR_OOM, ERR_STATE, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5, -6
NOALLOC_MAX_ELEMS = 4 * 1024 * 1024
IPC_EXPORT_BYTES = 256
OPT_SNAPSHOT, OPT_PROFILE, OPT_BF16_SHADOW, OPT_SWEEP = 1, 2, 3, 4
SNAPSHOT_COPY, SNAPSHOT_FLIP = 0, 1
KERNEL_LOCAL_STEP, KERNEL_SNAPSHOT, KERNEL_MEAN, KERNEL_MERGE = 0, 1, 2, 3
KERNEL_NAMES = {0: "local_step", 1: "snapshot", 2: "mean", 3: "merge", 4: "step_merge"}

_vp, _i, _i64, _f = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float

# name -> (restype, argtypes); must list every function include/cocod.h declares
SIGNATURES = {
    "cocod_create": (_i, [ctypes.POINTER(_vp), _i, _i64, _f, _f, _f]),
    "cocod_destroy": (_i, [_vp]),
    "cocod_local_step": (_i, [_vp, _vp]),
    "cocod_local_step_host": (_i, [_vp, _vp]),
    "cocod_comm_begin": (_i, [_vp, _vp]),
    "cocod_comm_end": (_i, [_vp]),
    "cocod_local_step_end": (_i, [_vp, _vp]),
    "cocod_local_sgd_average": (_i, [_vp]),
    "cocod_ssgd_step": (_i, [_vp, _vp]),
    "cocod_set_stream": (_i, [_vp, _vp]),
    "cocod_set_params": (_i, [_vp, _vp, _i]),
    "cocod_set_params_all": (_i, [_vp, _vp, _i]),
    "cocod_set_momentum": (_i, [_vp, _vp, _i]),
    "cocod_get_params": (_i, [_vp, _vp, _i]),
    "cocod_get_momentum": (_i, [_vp, _vp, _i]),
    "cocod_get_mean": (_i, [_vp, _vp, _i]),
    "cocod_get_bf16_shadow": (_i, [_vp, ctypes.POINTER(_vp)]),
    "cocod_set_lr": (_i, [_vp, _f]),
    "cocod_set_batch_sizes": (_i, [_vp, ctypes.POINTER(ctypes.c_double)]),
    "cocod_set_option": (_i, [_vp, _i, _i]),
    "cocod_sync": (_i, [_vp]),
    "cocod_comm_wait": (_i, [_vp, _i]),
    "cocod_step_count": (_i64, [_vp]),
    "cocod_last_cuda_error": (_i, [_vp]),
    "cocod_strerror": (ctypes.c_char_p, [_i]),
    "cocod_profile_reset": (_i, [_vp]),
    "cocod_profile_count": (_i, [_vp]),
    "cocod_profile_get": (_i, [_vp, _i, ctypes.POINTER(_i), ctypes.POINTER(_f), ctypes.POINTER(_f)]),
    "cocod_profile_get_device_ns": (_i, [_vp, _i, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]),
    "cocod_launch_count": (_i64, [_vp]),
    "cocod_set_shard": (_i, [_vp, _i, _i, ctypes.POINTER(ctypes.c_double)]),
    "cocod_mean_buffer": (_i, [_vp, ctypes.POINTER(_vp)]),
    "cocod_comm_exchanged": (_i, [_vp]),
    "cocod_ipc_export": (_i, [_vp, _vp]),
    "cocod_ipc_attach": (_i, [_vp, _i, _i, _vp]),
    "cocod_ipc_detach": (_i, [_vp]),
    "cocod_comm_gather": (_i, [_vp]),
    "cocod_kernel_mean_gather": (_i, [_vp, _i, _i64, _i64, _vp, _vp, _i, _i, _vp]),
    "cocod_kernel_local_step": (_i, [_vp, _vp, _vp, _vp, _i64, _f, _f, _f, _vp]),
    "cocod_kernel_snapshot": (_i, [_vp, _vp, _i64, _vp]),
    "cocod_kernel_mean": (_i, [_vp, _i, _i64, _vp, _vp, _vp]),
    "cocod_kernel_merge": (_i, [_vp, _vp, _vp, _i, _i64, _vp]),
    "cocod_kernel_local_step_host_noalloc": (_i, [_vp, _vp, _vp, _vp, _i64, _f, _f, _f, _vp]),
}

_lib = None


def load():
    """Load libcocod.so and declare every entry point.  Raises if the library is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing (no CPU fallback exists): build it with "
                               "`python -m paper_1906_12043_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class CocodError(RuntimeError):
    def __init__(self, code: int, where: str, cuda_error: int = 0):
        self.code = code
        msg = load().cocod_strerror(code).decode()
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{where}: {msg}{extra}")


def _ptr(t):
    """Device/host address of a torch tensor or numpy array (None -> NULL)."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(s):
    if s is None:
        return None
    return s.cuda_stream if hasattr(s, "cuda_stream") else int(s)


def _device_view(ptr: int, shape, dtype):
    """Wrap device memory owned by the library as a torch tensor (no copy, no ownership)."""
    import torch
    itemsize = torch.empty((), dtype=dtype).element_size()
    n = 1
    for d in shape:
        n *= int(d)

    class _Mem:
        __cuda_array_interface__ = {"shape": (n * itemsize,), "typestr": "|u1", "data": (int(ptr), False),
                                    "version": 2}

    return torch.as_tensor(_Mem(), device="cuda").view(dtype).view(*shape)


class Engine:
    """K workers x P parameters of CoCoD-SGD state in one GPU's HBM (see include/cocod.h)."""

    def __init__(self, K: int, P: int, lr: float, mu: float, wd: float, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the CoCoD-SGD engine needs a CUDA device (there is no CPU fallback)")
        self.K, self.P = int(K), int(P)
        self._lib = load()
        self._h = _vp()
        rc = self._lib.cocod_create(ctypes.byref(self._h), self.K, self.P, lr, mu, wd)
        if rc != OK:
            self._h = None
            raise CocodError(rc, "cocod_create")
        if stream is not None:
            self.set_stream(stream)

    # -- plumbing
    def _ck(self, rc: int, where: str):
        if rc != OK:
            raise CocodError(rc, where, self._lib.cocod_last_cuda_error(self._h) if self._h else 0)

    def _check_tensor(self, t, numel, name):
        import torch
        if isinstance(t, torch.Tensor):
            if t.dtype != torch.float32 or not t.is_contiguous() or t.numel() != numel:
                raise ValueError(f"{name}: need a contiguous float32 tensor of {numel} elements")
            return 0 if t.is_cuda else 1
        import numpy as np
        if not (isinstance(t, np.ndarray) and t.dtype == np.float32 and t.flags.c_contiguous and t.size == numel):
            raise ValueError(f"{name}: need a contiguous float32 array of {numel} elements")
        return 1

    def destroy(self):
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            self._lib.cocod_destroy(h)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- Algorithm 1
    def local_step(self, grads):
        """Step II, one iteration for all workers.  grads: K x P float32 CUDA tensor."""
        if self._check_tensor(grads, self.K * self.P, "grads") != 0:
            raise ValueError("grads must be a CUDA tensor (use local_step_host for host memory)")
        self._ck(self._lib.cocod_local_step(self._h, _ptr(grads)), "cocod_local_step")

    def local_step_host(self, grads):
        """Step II with the gradients in (pinned) host memory."""
        if self._check_tensor(grads, self.K * self.P, "grads") != 1:
            raise ValueError("grads must live in host memory")
        self._ck(self._lib.cocod_local_step_host(self._h, _ptr(grads)), "cocod_local_step_host")

    def comm_begin(self, side_stream=None):
        """Step I: store x_t^i and start the averaging on ``side_stream``."""
        self._ck(self._lib.cocod_comm_begin(self._h, _stream(side_stream)), "cocod_comm_begin")

    def local_step_end(self, grads):
        """The round's last local step and the merge in one pass (bit-identical to local_step + comm_end)."""
        if self._check_tensor(grads, self.K * self.P, "grads") != 0:
            raise ValueError("grads must be a CUDA tensor")
        self._ck(self._lib.cocod_local_step_end(self._h, _ptr(grads)), "cocod_local_step_end")

    def comm_end(self):
        """Line 6: x^i <- x_hat_t + (x^i - x_t^i)."""
        self._ck(self._lib.cocod_comm_end(self._h), "cocod_comm_end")

    # -- the sequential schemes of the paper's comparison
    def local_sgd_average(self):
        """Local-SGD's blocking model averaging: every x^i <- weighted mean of all x^j."""
        self._ck(self._lib.cocod_local_sgd_average(self._h), "cocod_local_sgd_average")

    def ssgd_step(self, grads):
        """S-SGD: average the K gradients, every worker applies the averaged gradient."""
        if self._check_tensor(grads, self.K * self.P, "grads") != 0:
            raise ValueError("grads must be a CUDA tensor")
        self._ck(self._lib.cocod_ssgd_step(self._h, _ptr(grads)), "cocod_ssgd_step")

    # -- around it
    def set_stream(self, stream):
        self._ck(self._lib.cocod_set_stream(self._h, _stream(stream)), "cocod_set_stream")

    def set_params(self, x0):
        self._ck(self._lib.cocod_set_params(self._h, _ptr(x0), self._check_tensor(x0, self.P, "x0")),
                 "cocod_set_params")

    def set_params_all(self, x):
        self._ck(self._lib.cocod_set_params_all(self._h, _ptr(x), self._check_tensor(x, self.K * self.P, "x")),
                 "cocod_set_params_all")

    def set_momentum(self, v):
        self._ck(self._lib.cocod_set_momentum(self._h, _ptr(v), self._check_tensor(v, self.K * self.P, "v")),
                 "cocod_set_momentum")

    def get_params(self, out=None):
        import torch
        if out is None:
            out = torch.empty((self.K, self.P), dtype=torch.float32, device="cuda")
        self._ck(self._lib.cocod_get_params(self._h, _ptr(out), self._check_tensor(out, self.K * self.P, "out")),
                 "cocod_get_params")
        return out

    def get_momentum(self, out=None):
        import torch
        if out is None:
            out = torch.empty((self.K, self.P), dtype=torch.float32, device="cuda")
        self._ck(self._lib.cocod_get_momentum(self._h, _ptr(out), self._check_tensor(out, self.K * self.P, "out")),
                 "cocod_get_momentum")
        return out

    def get_mean(self, out=None):
        import torch
        if out is None:
            out = torch.empty(self.P, dtype=torch.float32, device="cuda")
        self._ck(self._lib.cocod_get_mean(self._h, _ptr(out), self._check_tensor(out, self.P, "out")),
                 "cocod_get_mean")
        return out

    def bf16_shadow(self):
        """The engine's bf16 copy of x as a K x P torch.bfloat16 CUDA tensor (a view, no copy)."""
        import torch
        ptr = _vp()
        self._ck(self._lib.cocod_get_bf16_shadow(self._h, ctypes.byref(ptr)), "cocod_get_bf16_shadow")
        return _device_view(ptr.value, (self.K, self.P), torch.bfloat16)

    def set_lr(self, lr: float):
        self._ck(self._lib.cocod_set_lr(self._h, lr), "cocod_set_lr")

    def set_batch_sizes(self, M):
        if M is None:
            self._ck(self._lib.cocod_set_batch_sizes(self._h, None), "cocod_set_batch_sizes")
            return
        if len(M) != self.K:
            raise ValueError("need K batch sizes")
        arr = (ctypes.c_double * self.K)(*[float(m) for m in M])
        self._ck(self._lib.cocod_set_batch_sizes(self._h, arr), "cocod_set_batch_sizes")

    # -- workers spread over several GPUs (one engine per process)
    def set_shard(self, K_global: int, first: int, M_global=None):
        """This engine's K workers are workers first .. first+K-1 of K_global; M_global: the
        mini-batch sizes of ALL workers (None = equal).  K_global = 0 undoes it."""
        arr = None
        if M_global is not None:
            if len(M_global) != K_global:
                raise ValueError("need K_global batch sizes")
            arr = (ctypes.c_double * K_global)(*[float(m) for m in M_global])
        self._ck(self._lib.cocod_set_shard(self._h, int(K_global), int(first), arr), "cocod_set_shard")

    def mean_buffer(self):
        """The engine's average buffer as a torch CUDA tensor of P floats (a view, no copy): the
        operand of the caller's all-reduce."""
        import torch
        ptr = _vp()
        self._ck(self._lib.cocod_mean_buffer(self._h, ctypes.byref(ptr)), "cocod_mean_buffer")
        return _device_view(ptr.value, (self.P,), torch.float32)

    def comm_exchanged(self):
        self._ck(self._lib.cocod_comm_exchanged(self._h), "cocod_comm_exchanged")

    def ipc_export(self) -> bytes:
        buf = ctypes.create_string_buffer(IPC_EXPORT_BYTES)
        self._ck(self._lib.cocod_ipc_export(self._h, buf), "cocod_ipc_export")
        return buf.raw

    def ipc_attach(self, rank: int, blobs):
        """blobs: the ipc_export() bytes of all processes in rank order."""
        if any(len(b) != IPC_EXPORT_BYTES for b in blobs):
            raise ValueError("every blob must be IPC_EXPORT_BYTES long")
        raw = ctypes.create_string_buffer(b"".join(blobs), IPC_EXPORT_BYTES * len(blobs))
        self._ck(self._lib.cocod_ipc_attach(self._h, len(blobs), int(rank), raw), "cocod_ipc_attach")

    def ipc_detach(self):
        self._ck(self._lib.cocod_ipc_detach(self._h), "cocod_ipc_detach")

    def comm_gather(self):
        self._ck(self._lib.cocod_comm_gather(self._h), "cocod_comm_gather")

    def set_option(self, option: int, value: int):
        self._ck(self._lib.cocod_set_option(self._h, option, value), "cocod_set_option")

    def sync(self):
        self._ck(self._lib.cocod_sync(self._h), "cocod_sync")

    def comm_wait(self, timeout_ms: int) -> int:
        """Returns OK or ERR_TIMEOUT; raises on anything else."""
        rc = self._lib.cocod_comm_wait(self._h, int(timeout_ms))
        if rc not in (OK, ERR_TIMEOUT):
            self._ck(rc, "cocod_comm_wait")
        return rc

    @property
    def step_count(self) -> int:
        return int(self._lib.cocod_step_count(self._h))

    @property
    def launch_count(self) -> int:
        return int(self._lib.cocod_launch_count(self._h))

    # -- profiling
    def profile_reset(self):
        self._ck(self._lib.cocod_profile_reset(self._h), "cocod_profile_reset")

    def profile_records(self):
        """[(kind, start_ms, end_ms)] of every kernel since the last reset (syncs)."""
        n = self._lib.cocod_profile_count(self._h)
        if n < 0:
            self._ck(n, "cocod_profile_count")
        out = []
        kind, a, b = _i(), _f(), _f()
        for i in range(n):
            self._ck(self._lib.cocod_profile_get(self._h, i, ctypes.byref(kind), ctypes.byref(a), ctypes.byref(b)),
                     "cocod_profile_get")
            out.append((kind.value, a.value, b.value))
        return out

    def profile_device_records(self):
        """[(kind, start_ms, end_ms)] of the same records from the kernels' own stamps on the GPU's clock
        (milliseconds relative to the earliest stamp); records without stamps are left out."""
        n = self._lib.cocod_profile_count(self._h)
        if n < 0:
            self._ck(n, "cocod_profile_count")
        kind, a, b = _i(), _f(), _f()
        t0, t1 = ctypes.c_uint64(), ctypes.c_uint64()
        raw = []
        for i in range(n):
            self._ck(self._lib.cocod_profile_get(self._h, i, ctypes.byref(kind), ctypes.byref(a), ctypes.byref(b)),
                     "cocod_profile_get")
            self._ck(self._lib.cocod_profile_get_device_ns(self._h, i, ctypes.byref(t0), ctypes.byref(t1)),
                     "cocod_profile_get_device_ns")
            if t0.value and t1.value:
                raw.append((kind.value, t0.value, t1.value))
        if not raw:
            return []
        base = min(r[1] for r in raw)
        return [(k, (s - base) * 1e-6, (e - base) * 1e-6) for k, s, e in raw]


# ---------------------------------------------------------------------------------------------- stateless kernels
def _ck_rc(rc, where):
    if rc != OK:
        raise CocodError(rc, where)


def kernel_local_step(x_in, x_out, v, g, lr, mu, wd, stream=None):
    import torch
    s = _stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream
    _ck_rc(load().cocod_kernel_local_step(_ptr(x_in), _ptr(x_out), _ptr(v), _ptr(g), x_in.numel(), lr, mu, wd, s),
           "cocod_kernel_local_step")


def kernel_snapshot(x, snap, stream=None):
    import torch
    s = _stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream
    _ck_rc(load().cocod_kernel_snapshot(_ptr(x), _ptr(snap), x.numel(), s), "cocod_kernel_snapshot")


def kernel_mean(snap, mean, w=None, stream=None):
    import torch
    K, P = snap.shape
    s = _stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream
    _ck_rc(load().cocod_kernel_mean(_ptr(snap), K, P, _ptr(w), _ptr(mean), s), "cocod_kernel_mean")


def kernel_mean_gather(rows, col_lo, col_hi, outs, w=None, vec=4, stream=None):
    """rows: int64 CUDA tensor of K device addresses (one per worker's P stored values); outs: int64
    CUDA tensor of G device addresses of P-float average buffers; vec: columns per access (1, 4, 8)."""
    import torch
    s = _stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream
    _ck_rc(load().cocod_kernel_mean_gather(_ptr(rows), rows.numel(), int(col_lo), int(col_hi), _ptr(w), _ptr(outs),
                                           outs.numel(), int(vec), s), "cocod_kernel_mean_gather")


def kernel_merge(x, snap, mean, stream=None):
    import torch
    K, P = x.shape
    s = _stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream
    _ck_rc(load().cocod_kernel_merge(_ptr(x), _ptr(snap), _ptr(mean), K, P, s), "cocod_kernel_merge")


def kernel_local_step_host_noalloc(x_in, x_out, v, host_g, lr, mu, wd, stream=None):
    """Local step with host gradients for callers that must not allocate device memory: the
    gradients are staged through a fixed 16 MiB array inside the library (at most
    NOALLOC_MAX_ELEMS elements per call; larger requests raise with ERR_TOO_LARGE).  x_in, x_out,
    v: CUDA float32 tensors; host_g: float32 host tensor or array of the same element count."""
    import torch
    s = _stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream
    n = x_in.numel()
    count = host_g.numel() if hasattr(host_g, "numel") else host_g.size
    if count != n:
        raise ValueError("host_g must have as many elements as x_in")
    _ck_rc(load().cocod_kernel_local_step_host_noalloc(_ptr(x_in), _ptr(x_out), _ptr(v), _ptr(host_g), n,
                                                        lr, mu, wd, s), "cocod_kernel_local_step_host_noalloc")
