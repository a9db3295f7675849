"""CPU oracle of the per-worker stochastic gradient used by the end-to-end configuration --
TEST INFRASTRUCTURE ONLY (same rules as cocod_oracle.py: only tests, the smoke check and the
benchmark's CPU legs may import it; it imports nothing of the CUDA path).

Algorithm 1, Step II: each worker's stochastic gradient is the mean, over the M samples of its
mini-batch, of the per-sample gradients of f at its current model; here f = softmax cross-entropy
of a 3-layer ReLU MLP.  This is a textbook definition, so the
oracle is that definition written out in numpy fp64.  The workload stores weights in bfloat16
(fp32 master copy) and runs the contractions on tensor cores, so with ``emulate_bf16=True`` the
oracle rounds at exactly the points where the device path stores bfloat16:

    parameters used by forward/backward   bf16(master)            (all six tensors)
    h1, h2                                bf16(relu(z))
    dz3 = (softmax - onehot) / M          bf16
    dz2, dz1                              bf16(dh * (h > 0))
    every sum / product                   fp64 here (fp32 accumulation on the device)

With ``emulate_bf16=False`` nothing is rounded: that mode is what the pins check against finite
differences and against torch autograd.  The bf16-emulating mode differs from it only by the
``bf16`` calls, which are pinned separately (ties-to-even cases, torch's own conversion).
"""
from __future__ import annotations

import numpy as np


def bf16(a: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to the nearest bfloat16 (ties to even); returns fp64."""
    f = np.asarray(a, np.float64).astype(np.float32)      # fp64 -> fp32 first (as the device does)
    u = f.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def split(flat: np.ndarray, dims):
    d_in, d_h1, d_h2, d_out = dims
    shapes = [("W1", (d_h1, d_in)), ("b1", (d_h1,)), ("W2", (d_h2, d_h1)), ("b2", (d_h2,)),
              ("W3", (d_out, d_h2)), ("b3", (d_out,))]
    out, off = {}, 0
    for name, shape in shapes:
        n = int(np.prod(shape))
        out[name] = np.asarray(flat[off:off + n], np.float64).reshape(shape)
        off += n
    assert off == len(flat)
    return out


def loss_and_grad(flat: np.ndarray, X: np.ndarray, labels: np.ndarray, dims, emulate_bf16: bool = True,
                  return_preactivations: bool = False, flips=None, return_intermediates: bool = False):
    """Mean softmax cross-entropy of the minibatch and its gradient w.r.t. the flat parameters
    (same flat order).  Returns (loss fp64, grad fp32 array), plus the hidden pre-activations
    (z1, z2) on request: ReLU is a decision "z > 0", and a comparison against another precision is
    only meaningful for units whose |z| is not within rounding distance of 0.

    ``flips``: optional list of (layer, sample, unit) with layer 1 or 2: the ReLU decision of that unit
    for that sample is taken the OTHER way (on -> off: the activation and its gate are 0; off -> on: the
    gate is 1, the activation stays 0).  For a pre-activation within accumulation error of zero both
    outcomes are correct results of "z > 0" taken in finite precision; this lets a test evaluate the
    definition under the outcome another precision took.  The caller vouches that |z| is that small.

    ``return_intermediates``: the third return value is a dict of every intermediate of the definition
    (z1, z2, h1, h2, on1, on2, dz3, pre2 = dz3 W3, dz2, pre1 = dz2 W2, dz1) instead of (z1, z2)."""
    q = bf16 if emulate_bf16 else (lambda a: np.asarray(a, np.float64))
    p = {k: q(v) for k, v in split(flat, dims).items()}
    X = np.asarray(X, np.float64)
    M = X.shape[0]
    flip = {1: [], 2: []}
    for layer, b, j in (flips or []):
        flip[int(layer)].append((int(b), int(j)))

    def relu(z, which):
        """h = bf16(max(z, 0)) and the gate (h > 0), with the listed decisions taken the other way."""
        h = q(np.maximum(z, 0.0))
        on = h > 0
        for b, j in flip[which]:
            on[b, j] = not on[b, j]
            if not on[b, j]:
                h[b, j] = 0.0
        return h, on

    # forward
    z1 = X @ p["W1"].T + p["b1"]
    h1, on1 = relu(z1, 1)
    z2 = h1 @ p["W2"].T + p["b2"]
    h2, on2 = relu(z2, 2)
    z3 = h2 @ p["W3"].T + p["b3"]
    zmax = z3.max(axis=1, keepdims=True)
    e = np.exp(z3 - zmax)
    s = e.sum(axis=1, keepdims=True)
    loss = float(np.mean(np.log(s[:, 0]) + zmax[:, 0] - z3[np.arange(M), labels]))
    # backward
    onehot = np.zeros_like(z3)
    onehot[np.arange(M), labels] = 1.0
    dz3 = q((e / s - onehot) / M)
    g = {"W3": dz3.T @ h2, "b3": dz3.sum(0)}
    pre2 = dz3 @ p["W3"]
    dz2 = q(pre2 * on2)
    g["W2"], g["b2"] = dz2.T @ h1, dz2.sum(0)
    pre1 = dz2 @ p["W2"]
    dz1 = q(pre1 * on1)
    g["W1"], g["b1"] = dz1.T @ X, dz1.sum(0)
    flat_g = np.concatenate([g[k].ravel() for k in ("W1", "b1", "W2", "b2", "W3", "b3")])
    if return_intermediates:
        return loss, flat_g.astype(np.float32), dict(z1=z1, z2=z2, h1=h1, h2=h2, on1=on1, on2=on2, dz3=dz3, pre2=pre2,
                                                     dz2=dz2, pre1=pre1, dz1=dz1)
    if return_preactivations:
        return loss, flat_g.astype(np.float32), (z1, z2)
    return loss, flat_g.astype(np.float32)
