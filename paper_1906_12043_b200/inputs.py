"""Seeded synthetic inputs for the CoCoD-SGD parameter engine.

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests/bench.  It holds NO arithmetic of the method (no SGD step, no
mean, no merge): it only produces the initial point and the per-(worker, step)
stochastic gradients that the method consumes as inputs.

The paper's workloads are CIFAR trainings of ResNet18 / VGG16 (Section 5.1);
the engine's cost and arithmetic depend only on the number of workers K (the
paper's N), the flattened model size P (the paper's d) and the period k, so
i.i.d. Gaussian vectors of those sizes stand in for real gradients.

Generator (counter based, random access, identical on host and device):

    key  = fold(seed, stream, worker, step)          four rounds of a 64-bit mixer
    h    = mix64(key + (p + 1) * GOLDEN)              one 64-bit word per element
    u1   = ((h >> 32) + 1) / 2**32   in (0, 1]
    u2   = (h & 0xffffffff) / 2**32  in [0, 1)
    z    = sqrt(-2 ln u1) * cos(2 pi u2)              Box-Muller, cosine branch
    out  = float32(sigma * z)

``ln`` and ``cos`` are NOT library calls: they are fixed polynomial recipes
built only from IEEE-754 double add / multiply / divide / sqrt in a fixed order
with no fused multiply-add, so the numpy implementation below and the CUDA
implementation in ``csrc/inputs_gen.cu`` return the same bits.  (Whatever the
recipe returns *is* the definition of the input; its accuracy, about 1e-16, only
has to make the values Gaussian.)
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

MASK64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15
MIX_A = 0xBF58476D1CE4E5B9
MIX_B = 0x94D049BB133111EB

# stream ids: which family of numbers a key belongs to
STREAM_X0 = 1       # initial point, worker = 0, step = 0
STREAM_GRAD = 2     # stochastic gradient of (worker, step)
STREAM_DATA = 3     # MLP minibatch inputs of (worker, step)
STREAM_WEIGHT = 4   # MLP weight init (worker field = tensor index)

LN2 = 0.6931471805599453
SQRT_HALF = 0.7071067811865476
PI_4 = 0.7853981633974483

# atanh series 1/(2n+1), n = 10 .. 0 (Horner order)
_LN_COEF = [1.0 / (2 * n + 1) for n in range(10, -1, -1)]
# sin(y)/y = sum (-1)^n y^(2n)/(2n+1)!, n = 7 .. 0 ; cos(y) = sum (-1)^n y^(2n)/(2n)!, n = 8 .. 0
_FACT = [1.0]
for _i in range(1, 18):
    _FACT.append(_FACT[-1] * _i)
_SIN_COEF = [((-1.0) ** n) / _FACT[2 * n + 1] for n in range(7, -1, -1)]
_COS_COEF = [((-1.0) ** n) / _FACT[2 * n] for n in range(8, -1, -1)]


def mix64_int(z: int) -> int:
    """64-bit finaliser (splitmix64's output function) on a Python int."""
    z &= MASK64
    z = ((z ^ (z >> 30)) * MIX_A) & MASK64
    z = ((z ^ (z >> 27)) * MIX_B) & MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int, worker: int, step: int) -> int:
    """Fold the four counters into one 64-bit key."""
    k = mix64_int(seed + GOLDEN)
    k = mix64_int(k + stream)
    k = mix64_int(k + worker)
    k = mix64_int(k + step)
    return k


def _mix64_np(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * np.uint64(MIX_A)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(MIX_B)
    return z ^ (z >> np.uint64(31))


def element_bits(key: int, p: np.ndarray) -> np.ndarray:
    """The 64-bit word of element index p (uint64 array) under ``key``."""
    with np.errstate(over="ignore"):
        z = np.uint64(key) + (p.astype(np.uint64) + np.uint64(1)) * np.uint64(GOLDEN)
        return _mix64_np(z)


def std_normal_from_bits(h: np.ndarray) -> np.ndarray:
    """Box-Muller on a uint64 array -> float64 standard normals (fixed recipe)."""
    a = (h >> np.uint64(32)) + np.uint64(1)            # 1 .. 2**32
    b = h & np.uint64(0xFFFFFFFF)
    # ---- ln(u1), u1 = a / 2**32 : a = f * 2**E, f in [0.5, 1)
    f, E = np.frexp(a.astype(np.float64))
    low = f < SQRT_HALF
    f = np.where(low, f * 2.0, f)                      # f in [sqrt(.5), sqrt(2))
    E = np.where(low, E - 1, E)
    s = (f - 1.0) / (f + 1.0)
    s2 = s * s
    poly = np.full_like(s2, _LN_COEF[0])
    for c in _LN_COEF[1:]:
        poly = poly * s2 + c
    ln_f = (2.0 * s) * poly
    ln_u1 = (E - 32).astype(np.float64) * LN2 + ln_f
    r = np.sqrt(-2.0 * ln_u1)
    # ---- cos(2 pi u2), u2 = b / 2**32 : octant o, remainder rem / 2**29 of an octant
    o = (b >> np.uint64(29)).astype(np.int64)
    rem = (b & np.uint64((1 << 29) - 1)).astype(np.int64)
    odd = (o & 1) == 1
    rem = np.where(odd, (1 << 29) - rem, rem)
    y = (rem.astype(np.float64) * (1.0 / (1 << 29))) * PI_4     # in [0, pi/4]
    y2 = y * y
    ps = np.full_like(y2, _SIN_COEF[0])
    for c in _SIN_COEF[1:]:
        ps = ps * y2 + c
    ps = ps * y
    pc = np.full_like(y2, _COS_COEF[0])
    for c in _COS_COEF[1:]:
        pc = pc * y2 + c
    use_sin = (o == 1) | (o == 2) | (o == 5) | (o == 6)
    neg = (o >= 2) & (o <= 5)
    c = np.where(use_sin, ps, pc)
    c = np.where(neg, -c, c)
    return r * c


def gaussian(seed: int, stream: int, worker: int, step: int, p0: int, n: int,
             sigma: float, chunk: int = 1 << 16) -> np.ndarray:
    """float32 values sigma*Z for element indices p0 .. p0+n-1 (host, numpy)."""
    key = stream_key(seed, stream, worker, step)
    out = np.empty(n, dtype=np.float32)
    for c0 in range(0, n, chunk):
        c1 = min(n, c0 + chunk)
        p = np.arange(p0 + c0, p0 + c1, dtype=np.uint64)
        out[c0:c1] = (sigma * std_normal_from_bits(element_bits(key, p))).astype(np.float32)
    return out


def gaussian_at(seed: int, stream: int, worker: int, step: int, cols: np.ndarray,
                sigma: float) -> np.ndarray:
    """float32 values sigma*Z at the given element indices (any order)."""
    key = stream_key(seed, stream, worker, step)
    p = np.asarray(cols, dtype=np.uint64)
    return (sigma * std_normal_from_bits(element_bits(key, p))).astype(np.float32)


# ----------------------------------------------------------------------------- workload recipes
X0_SEED = 0        # "seed 0" of the configs
GRAD_SEED = 1234   # free choice, fixed here


def initial_point(P: int, sigma: float = 0.01, seed: int = X0_SEED, cols=None) -> np.ndarray:
    """x0 of length P (or at ``cols``): the same vector for every worker."""
    if cols is not None:
        return gaussian_at(seed, STREAM_X0, 0, 0, cols, sigma)
    return gaussian(seed, STREAM_X0, 0, 0, 0, P, sigma)


def gradients(K: int, P: int, step: int, sigma: float = 0.01, seed: int = GRAD_SEED,
              cols=None) -> np.ndarray:
    """K x P (or K x len(cols)) float32 gradients of global local-step index ``step``."""
    if cols is not None:
        return np.stack([gaussian_at(seed, STREAM_GRAD, w, step, cols, sigma) for w in range(K)])
    return np.stack([gaussian(seed, STREAM_GRAD, w, step, 0, P, sigma) for w in range(K)])


def shard_columns(P_total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous column range [lo, hi) of ``rank``; ranges tile [0, P_total) and
    every boundary is a multiple of 64 elements (256 B) except the last."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    blocks = (P_total + 63) // 64
    lo_b = (blocks * rank) // world
    hi_b = (blocks * (rank + 1)) // world
    return min(P_total, lo_b * 64), min(P_total, hi_b * 64)


# ----------------------------------------------------------------------------- device generator
_LIB = None


def _lib():
    """The CUDA build of the same generator (its own shared library, not the engine's)."""
    global _LIB
    if _LIB is None:
        path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcocod_inputs.so")
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -c 'import __graft_entry__ as g; g.build()'`")
        lib = ctypes.CDLL(path)
        lib.cocod_inputs_gaussian_f32.restype = ctypes.c_int
        lib.cocod_inputs_gaussian_f32.argtypes = [
            ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_double, ctypes.c_void_p]
        lib.cocod_inputs_gaussian_bf16.restype = ctypes.c_int
        lib.cocod_inputs_gaussian_bf16.argtypes = lib.cocod_inputs_gaussian_f32.argtypes
        _LIB = lib
    return _LIB


def device_gaussian_into(out, seed: int, stream: int, worker: int, step: int, p0: int,
                         sigma: float, cuda_stream: int = 0) -> None:
    """Fill a contiguous float32 (or bfloat16) CUDA tensor ``out`` with sigma*Z for
    indices p0 .. p0+out.numel()-1 on the given CUDA stream (0 = torch's current)."""
    import torch
    if not out.is_cuda or not out.is_contiguous():
        raise ValueError("device_gaussian_into needs a contiguous CUDA tensor")
    if cuda_stream == 0:
        cuda_stream = torch.cuda.current_stream(out.device).cuda_stream
    key = stream_key(seed, stream, worker, step)
    lib = _lib()
    if out.dtype == torch.float32:
        fn = lib.cocod_inputs_gaussian_f32
    elif out.dtype == torch.bfloat16:
        fn = lib.cocod_inputs_gaussian_bf16
    else:
        raise ValueError("float32 or bfloat16 only")
    with torch.cuda.device(out.device):
        rc = fn(out.data_ptr(), key, p0, out.numel(), sigma, cuda_stream)
    if rc != 0:
        raise RuntimeError(f"cocod_inputs_gaussian failed: cuda error {rc}")


def device_gradients_into(g, step: int, sigma: float = 0.01, seed: int = GRAD_SEED,
                          p0: int = 0, first_worker: int = 0) -> None:
    """Fill a K x P float32 CUDA tensor with the gradients of local step ``step``
    (columns p0 .. p0+P-1 of the global vector, workers first_worker .. first_worker+K-1)."""
    K = g.shape[0]
    for w in range(K):
        device_gaussian_into(g[w], seed, STREAM_GRAD, first_worker + w, step, p0, sigma)


# ----------------------------------------------------------------------------- synthetic MLP workload
# End-to-end configuration: every worker trains a 3-layer ReLU MLP (784 -> 1024 -> 1024 -> 10) on
# minibatches of 128 Gaussian inputs whose labels come from a fixed random "teacher" MLP of the
# same shape.  Flat parameter order: W1, b1, W2, b2, W3, b3, each W row-major [out][in].
MLP_DIMS = (784, 1024, 1024, 10)
MLP_BATCH = 128
MLP_STUDENT_SEED, MLP_TEACHER_SEED, MLP_DATA_SEED = 0, 1, 2


def mlp_segments(dims=MLP_DIMS):
    """[(name, offset, shape)] of the flat parameter vector, and its length P."""
    d_in, d_h1, d_h2, d_out = dims
    segs, off = [], 0
    for name, shape in (("W1", (d_h1, d_in)), ("b1", (d_h1,)), ("W2", (d_h2, d_h1)), ("b2", (d_h2,)),
                        ("W3", (d_out, d_h2)), ("b3", (d_out,))):
        n = int(np.prod(shape))
        segs.append((name, off, shape))
        off += n
    return segs, off


def mlp_init_params(seed: int, dims=MLP_DIMS) -> np.ndarray:
    """Flat fp32 parameters: W ~ N(0, 1/fan_in), b = 0."""
    segs, P = mlp_segments(dims)
    out = np.zeros(P, np.float32)
    for t, (name, off, shape) in enumerate(segs):
        if name.startswith("W"):
            n = int(np.prod(shape))
            out[off:off + n] = gaussian(seed, STREAM_WEIGHT, t, 0, 0, n, 1.0 / np.sqrt(shape[1]))
    return out


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array -> the nearest bfloat16 values (ties to even), returned as float32."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 values that are exactly representable in bfloat16 -> their 16-bit patterns."""
    return (np.ascontiguousarray(a, np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def mlp_batch(worker: int, step: int, batch: int = MLP_BATCH, d_in: int = MLP_DIMS[0],
              seed: int = MLP_DATA_SEED) -> np.ndarray:
    """Minibatch of (worker, step): batch x d_in values ~ N(0, 1), rounded once to bfloat16."""
    x = gaussian(seed, STREAM_DATA, worker, step, 0, batch * d_in, 1.0)
    return round_to_bf16(x).reshape(batch, d_in)


def mlp_teacher_labels(X: np.ndarray, teacher: np.ndarray, dims=MLP_DIMS) -> np.ndarray:
    """Labels of a minibatch: argmax of the teacher MLP's logits, computed once on the host in
    fp64 and handed to both sides (never recomputed on the GPU, so near-ties cannot flip)."""
    segs, _ = mlp_segments(dims)
    p = {name: teacher[off:off + int(np.prod(shape))].astype(np.float64).reshape(shape)
         for name, off, shape in segs}
    h = np.maximum(X.astype(np.float64) @ p["W1"].T + p["b1"], 0.0)
    h = np.maximum(h @ p["W2"].T + p["b2"], 0.0)
    return np.argmax(h @ p["W3"].T + p["b3"], axis=1).astype(np.int32)


def device_mlp_batches_into(out, first_step: int, seed: int = MLP_DATA_SEED) -> None:
    """Fill a CUDA bfloat16 tensor [steps][K][batch][d_in] with the minibatches of global steps
    first_step .. first_step + steps - 1 (the same bytes as ``mlp_batch`` gives on the host)."""
    steps, K = out.shape[0], out.shape[1]
    for t in range(steps):
        for w in range(K):
            device_gaussian_into(out[t, w], seed, STREAM_DATA, w, first_step + t, 0, 1.0)


def device_mlp_teacher_labels(X, teacher: np.ndarray, dims=MLP_DIMS, rows_per_pass: int = 1 << 16):
    """Labels of minibatches held on the device: argmax of the teacher MLP's logits in fp64 (torch on the
    device; the same definition as ``mlp_teacher_labels``).  X: CUDA bfloat16 [..., d_in]; returns int32
    [...].  Whoever compares two implementations hands BOTH this one array (a near-tie could fall
    differently under another summation order)."""
    import torch
    segs, _ = mlp_segments(dims)
    p = {name: torch.from_numpy(teacher[off:off + int(np.prod(shape))].astype(np.float64).reshape(shape)).to(X.device)
         for name, off, shape in segs}
    flat = X.reshape(-1, X.shape[-1])
    out = torch.empty(flat.shape[0], dtype=torch.int32, device=X.device)
    for r0 in range(0, flat.shape[0], rows_per_pass):
        h = torch.relu(flat[r0:r0 + rows_per_pass].double() @ p["W1"].T + p["b1"])
        h = torch.relu(h @ p["W2"].T + p["b2"])
        out[r0:r0 + rows_per_pass] = torch.argmax(h @ p["W3"].T + p["b3"], dim=1).to(torch.int32)
    return out.reshape(X.shape[:-1])
