"""CPU oracle of CoCoD-SGD's parameter path -- TEST INFRASTRUCTURE ONLY.

A sequential restatement of Algorithm 1 of the paper: the element loops are the
plain C of ``cocod_oracle.c`` (compiled here with gcc on first use), the round
structure is the Python below.  Only ``tests/``, the smoke check and the
benchmark's CPU-baseline leg may import this; the CUDA library and its binding
never do, and this file imports nothing of theirs.

Modes (see the C file's header): ``"ref"`` fp32-stored / fp64-evaluated (the
parity target), ``"f64"`` fp64 state, ``"mirror"`` pure fp32 in a fixed
operation order (bit-exact twin of a device kernel that keeps that order).
No function here is unpinned: tests/test_oracle_pins.py ties each to closed
forms, invariants, hand-computed rounds and an exact-rational brute force.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cocod_oracle.c")
_SO = os.path.join(_HERE, "libcocod_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (plain gcc, -O2, no contraction, OpenMP for the timed baseline)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fPIC",
                               "-shared", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        i, i64, f, d = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_double
        for name in ("oracle_local_step_ref", "oracle_local_step_mirror"):
            getattr(L, name).argtypes = [i, i64, f32p, f32p, f32p, f, f, f]
        L.oracle_local_step_f64.argtypes = [i, i64, f64p, f64p, f64p, d, d, d]
        L.oracle_snapshot_f32.argtypes = [i, i64, f32p, f32p]
        L.oracle_snapshot_f64.argtypes = [i, i64, f64p, f64p]
        for name in ("oracle_mean_ref", "oracle_mean_mirror"):
            getattr(L, name).argtypes = [i, i64, f32p, f64p, f32p]
        L.oracle_mean_f64.argtypes = [i, i64, f64p, f64p, f64p]
        for name in ("oracle_merge_ref", "oracle_merge_mirror"):
            getattr(L, name).argtypes = [i, i64, f32p, f32p, f32p]
        L.oracle_merge_f64.argtypes = [i, i64, f64p, f64p, f64p]
        L.oracle_set_threads.argtypes = [i]
        L.oracle_get_threads.restype = i
        L.oracle_max_threads.restype = i
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def _p(a: np.ndarray):
    if a.dtype == np.float32:
        return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


class OracleEngine:
    """Algorithm 1 over K workers held as the rows of K x P arrays.

    The call sequence is the algorithm's: ``comm_begin`` is Step I (store x_t^i, form the
    weighted mean of the stored copies), ``local_step`` is one iteration of Step II,
    ``comm_end`` is line 6.  Running Step I concurrently with Step II changes no value (the
    mean reads only the stored copies), so this oracle simply does Step I at once.

    ``batch_sizes`` are the M_i of Algorithm 1 (None = all equal).  Hyper-parameters are taken
    as fp32 values, because that is what the C boundary of the engine carries.
    """

    def __init__(self, K: int, P: int, lr: float, mu: float, wd: float, mode: str = "ref",
                 batch_sizes=None):
        if mode not in ("ref", "f64", "mirror"):
            raise ValueError(mode)
        self.K, self.P, self.mode = int(K), int(P), mode
        self.lr, self.mu, self.wd = np.float32(lr), np.float32(mu), np.float32(wd)
        self.dt = np.float64 if mode == "f64" else np.float32
        self.x = np.zeros((K, P), self.dt)
        self.v = np.zeros((K, P), self.dt)
        self.snap = np.zeros((K, P), self.dt)
        self.mean = np.zeros(P, self.dt)
        self.M = None if batch_sizes is None else np.ascontiguousarray(batch_sizes, np.float64)
        self.in_flight = False
        self.steps = 0

    # -- Initialize: x_i^0 = x_hat_0 for every worker (Algorithm 1, "Initialize")
    def set_params(self, x0) -> None:
        self.x[:] = np.asarray(x0, self.dt)[None, :]

    def set_params_all(self, x) -> None:
        self.x[:] = np.asarray(x, self.dt)

    def set_lr(self, lr: float) -> None:
        self.lr = np.float32(lr)

    # -- Step II, one iteration
    def local_step(self, g) -> None:
        g = np.ascontiguousarray(g, self.dt)
        assert g.shape == (self.K, self.P)
        L = lib()
        if self.mode == "ref":
            L.oracle_local_step_ref(self.K, self.P, _p(self.x), _p(self.v), _p(g), self.lr, self.mu, self.wd)
        elif self.mode == "mirror":
            L.oracle_local_step_mirror(self.K, self.P, _p(self.x), _p(self.v), _p(g), self.lr, self.mu, self.wd)
        else:
            L.oracle_local_step_f64(self.K, self.P, _p(self.x), _p(self.v), _p(g),
                                    float(self.lr), float(self.mu), float(self.wd))
        self.steps += 1

    # -- Step I
    def comm_begin(self) -> None:
        if self.in_flight:
            raise RuntimeError("communication already in flight")
        L = lib()
        Mp = None if self.M is None else _p(self.M)
        if self.mode == "f64":
            L.oracle_snapshot_f64(self.K, self.P, _p(self.x), _p(self.snap))
            L.oracle_mean_f64(self.K, self.P, _p(self.snap), Mp, _p(self.mean))
        else:
            L.oracle_snapshot_f32(self.K, self.P, _p(self.x), _p(self.snap))
            fn = L.oracle_mean_ref if self.mode == "ref" else L.oracle_mean_mirror
            fn(self.K, self.P, _p(self.snap), Mp, _p(self.mean))
        self.in_flight = True

    # -- line 6
    def comm_end(self) -> None:
        if not self.in_flight:
            raise RuntimeError("no communication in flight")
        L = lib()
        if self.mode == "f64":
            L.oracle_merge_f64(self.K, self.P, _p(self.x), _p(self.snap), _p(self.mean))
        elif self.mode == "ref":
            L.oracle_merge_ref(self.K, self.P, _p(self.x), _p(self.snap), _p(self.mean))
        else:
            L.oracle_merge_mirror(self.K, self.P, _p(self.x), _p(self.snap), _p(self.mean))
        self.in_flight = False

    # -- the sequential schemes the paper compares against (Section 2; Section 4.2)
    def local_sgd_average(self) -> None:
        """Local-SGD: every worker's model becomes the weighted mean of all models."""
        if self.in_flight:
            raise RuntimeError("communication in flight")
        L = lib()
        Mp = None if self.M is None else _p(self.M)
        fn = {"ref": L.oracle_mean_ref, "mirror": L.oracle_mean_mirror, "f64": L.oracle_mean_f64}[self.mode]
        fn(self.K, self.P, _p(self.x), Mp, _p(self.mean))
        self.x[:] = self.mean[None, :]

    def ssgd_step(self, g) -> None:
        """S-SGD: the workers' gradients are averaged with the same weights and every worker applies
        the averaged gradient (equivalent to one worker with the summed mini-batch)."""
        if self.in_flight:
            raise RuntimeError("communication in flight")
        g = np.ascontiguousarray(g, self.dt)
        L = lib()
        Mp = None if self.M is None else _p(self.M)
        gbar = np.zeros(self.P, self.dt)
        fn = {"ref": L.oracle_mean_ref, "mirror": L.oracle_mean_mirror, "f64": L.oracle_mean_f64}[self.mode]
        fn(self.K, self.P, _p(g), Mp, _p(gbar))
        self.local_step(np.ascontiguousarray(np.tile(gbar, (self.K, 1))))

    def run(self, grad_fn, k: int, rounds: int, on_round=None) -> None:
        """The while loop of Algorithm 1 for whole rounds: ``grad_fn(tau)`` returns the
        K x P gradients of global local-step index tau = round * k + s."""
        for r in range(rounds):
            self.comm_begin()
            for s in range(k):
                self.local_step(grad_fn(r * k + s))
            self.comm_end()
            if on_round is not None:
                on_round(r, self)
