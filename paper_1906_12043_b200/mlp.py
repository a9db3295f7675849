"""Thin ctypes binding over the MLP-gradient entry points of libcocod.so (include/cocod_mlp.h).

Marshalling only: the gradients are computed by the library's CUDA kernels (tcgen05 GEMMs and
small fused kernels).  No CPU fallback.
"""
from __future__ import annotations

import ctypes

from . import engine as _E

_vp, _i, _i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64

SIGNATURES = {
    "cocod_mlp_create": (_i, [ctypes.POINTER(_vp), _i, _i, _i, _i, _i]),
    "cocod_mlp_destroy": (_i, [_vp]),
    "cocod_mlp_param_count": (_i64, [_vp]),
    "cocod_mlp_param_count_unpadded": (_i64, [_vp]),
    "cocod_mlp_grad": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "cocod_mlp_grad_step": (_i, [_vp, _vp, _vp, _vp, _vp]),
    "cocod_mlp_check": (_i, [_vp, _vp]),
    "cocod_mlp_set_option": (_i, [_vp, _i, _i]),
    "cocod_mlp_profile_get": (_i, [_vp, ctypes.POINTER(_i), ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]),
    "cocod_mlp_profile_get_device": (_i, [_vp, ctypes.POINTER(_i), ctypes.POINTER(ctypes.c_float)]),
    "cocod_mlp_launch_count": (_i64, [_vp]),
    "cocod_gemm_wait_selftest": (_i, [_i, _vp]),
    "cocod_gemm_update_wait_selftest": (_i, [_i, _vp]),
    "cocod_mlp_chain_wait_selftest": (_i, [_i, _vp]),
    "cocod_gemm_bf16": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i64, _i64, _i64, _i64, _i64, _i64, _vp]),
}

OPT_PROFILE = 1
OPT_CHAIN = 2
_declared = False


def load():
    global _declared
    lib = _E.load()
    if not _declared:
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _declared = True
    return lib


def _cur_stream(stream):
    import torch
    return _E._stream(stream) if stream is not None else torch.cuda.current_stream().cuda_stream


class MLPGrad:
    """Batched mini-batch gradients of the 3-layer ReLU MLP for K workers."""

    def __init__(self, K: int, batch: int = 128, d_in: int = 784, d_hidden: int = 1024, d_out: int = 10):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the MLP gradient path needs a CUDA device (there is no CPU fallback)")
        self._lib = load()
        self._h = _vp()
        rc = self._lib.cocod_mlp_create(ctypes.byref(self._h), K, batch, d_in, d_hidden, d_out)
        if rc != _E.OK:
            self._h = None
            raise _E.CocodError(rc, "cocod_mlp_create")
        self.K, self.batch, self.dims = K, batch, (d_in, d_hidden, d_hidden, d_out)
        self.P = int(self._lib.cocod_mlp_param_count(self._h))
        self.P_raw = int(self._lib.cocod_mlp_param_count_unpadded(self._h))

    def grad(self, params_bf16, x, labels, grads, loss, stream=None):
        """params_bf16: K x P bf16; x: K x batch x d_in bf16; labels: K x batch int32;
        grads: K x P fp32 (out); loss: K fp32 (out).  All CUDA tensors, contiguous."""
        import torch
        K, P, B, d_in = self.K, self.P, self.batch, self.dims[0]
        for t, dt, n, nm in ((params_bf16, torch.bfloat16, K * P, "params_bf16"), (x, torch.bfloat16, K * B * d_in, "x"),
                             (labels, torch.int32, K * B, "labels"), (grads, torch.float32, K * P, "grads"),
                             (loss, torch.float32, K, "loss")):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == dt and t.numel() == n):
                raise ValueError(f"{nm}: need a contiguous CUDA {dt} tensor of {n} elements")
        rc = self._lib.cocod_mlp_grad(self._h, params_bf16.data_ptr(), x.data_ptr(), labels.data_ptr(),
                                      grads.data_ptr(), loss.data_ptr(), _cur_stream(stream))
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_grad")

    def grad_step(self, engine, x, labels, loss):
        """Gradients and the engine's local step in one call (a persistent kernel forms the weight
        gradients of W1 and W2 tile by tile and updates each tile at once).  ``engine``: an Engine with K x P matching and the
        bf16 shadow switched on.  Bit-identical to grad(...) followed by engine.local_step(grads)."""
        import torch
        K, B, d_in = self.K, self.batch, self.dims[0]
        for t, dt, n, nm in ((x, torch.bfloat16, K * B * d_in, "x"), (labels, torch.int32, K * B, "labels"),
                             (loss, torch.float32, K, "loss")):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == dt and t.numel() == n):
                raise ValueError(f"{nm}: need a contiguous CUDA {dt} tensor of {n} elements")
        rc = self._lib.cocod_mlp_grad_step(self._h, engine._h, x.data_ptr(), labels.data_ptr(), loss.data_ptr())
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_grad_step")

    def check(self, stream=None):
        rc = self._lib.cocod_mlp_check(self._h, _cur_stream(stream))
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_check")

    def set_profile(self, on):
        """0 / False: off; 1 / True: CUDA events around each pass and the update kernel; 2: the update kernel's own
        time stamps only (nothing about the launches changes)."""
        rc = self._lib.cocod_mlp_set_option(self._h, OPT_PROFILE, int(on))
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_set_option")

    def set_chain(self, on):
        """True (default): the part of a pass before the weight gradients (both hidden layers, the output layer, the
        hidden deltas) runs as one kernel whose thread blocks hand tiles to one another through counters in global
        memory; False: one kernel per layer.  Both give the same bits."""
        rc = self._lib.cocod_mlp_set_option(self._h, OPT_CHAIN, 1 if on else 0)
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_set_option")

    def profile(self):
        """(recorded calls, average ms of a whole gradient pass, average ms of the gradient + update kernel)."""
        n, a, b = _i(), ctypes.c_float(), ctypes.c_float()
        rc = self._lib.cocod_mlp_profile_get(self._h, ctypes.byref(n), ctypes.byref(a), ctypes.byref(b))
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_profile_get")
        return n.value, a.value, b.value

    def profile_device(self):
        """(stamped launches of the gradient + update kernel, their average ms by the kernel's own stamps)."""
        n, a = _i(), ctypes.c_float()
        rc = self._lib.cocod_mlp_profile_get_device(self._h, ctypes.byref(n), ctypes.byref(a))
        if rc != _E.OK:
            raise _E.CocodError(rc, "cocod_mlp_profile_get_device")
        return n.value, a.value

    @property
    def launch_count(self) -> int:
        return int(self._lib.cocod_mlp_launch_count(self._h))

    def destroy(self):
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            self._lib.cocod_mlp_destroy(h)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def gemm_bf16(A, B, C, a_rows_contiguous=False, b_rows_contiguous=False, stream=None):
    """C[w][m][n] = sum_k A_w(m, k) B_w(n, k) for CUDA tensors: A is W x M x K (or W x K x M when
    a_rows_contiguous), B is W x N x K (or W x K x N when b_rows_contiguous), both bf16; C is
    W x M x N fp32."""
    W, M, N = C.shape
    K = A.shape[1] if a_rows_contiguous else A.shape[2]
    rc = load().cocod_gemm_bf16(A.data_ptr(), B.data_ptr(), C.data_ptr(), M, N, K, W, int(a_rows_contiguous),
                                int(b_rows_contiguous), A.stride(1), B.stride(1), C.stride(1), A.stride(0),
                                B.stride(0), C.stride(0), _cur_stream(stream))
    if rc != _E.OK:
        raise _E.CocodError(rc, "cocod_gemm_bf16")


def gemm_update_wait_selftest(wait_ms: int = 50, stream=None) -> int:
    """The bounded-wait self-test of the persistent gradient + update kernel (ERR_TIMEOUT is the expected code)."""
    return int(load().cocod_gemm_update_wait_selftest(int(wait_ms), _cur_stream(stream)))


def chain_wait_selftest(wait_ms: int = 50, stream=None) -> int:
    """The bounded-wait self-test of the chain kernel (ERR_TIMEOUT is the expected code)."""
    return int(load().cocod_mlp_chain_wait_selftest(int(wait_ms), _cur_stream(stream)))


def gemm_wait_selftest(wait_ms: int = 50, stream=None) -> int:
    """Run the bounded-wait self-test; returns the library's code (ERR_TIMEOUT is the expected one)."""
    return int(load().cocod_gemm_wait_selftest(int(wait_ms), _cur_stream(stream)))
