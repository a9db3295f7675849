"""The process pool that computes the K workers' oracle gradients for the end-to-end run (tests/c4_loss_curve.py)
must return exactly what the oracle returns in-process: same minibatch bytes, labels, losses and gradients."""
import numpy as np

import c4_loss_curve as C
from oracle import mlp_oracle as MO
from paper_1906_12043_b200 import inputs as I


def test_pooled_oracle_gradients_equal_the_in_process_oracle():
    K, tau = 2, 6
    loop = C.OracleLoop(K, 0.05, 0.9, 0.0, procs=2)
    try:
        loop.eng.set_params(I.mlp_init_params(I.MLP_STUDENT_SEED))
        losses, Xb, y, flips = loop.gradients(tau)
        assert flips == []
        teacher = I.mlp_init_params(I.MLP_TEACHER_SEED)
        for w in range(K):
            X = I.mlp_batch(w, tau)
            yy = I.mlp_teacher_labels(X, teacher)
            ll, g = MO.loss_and_grad(loop.eng.x[w], X, yy, I.MLP_DIMS)
            assert np.array_equal(g, loop.g[w]) and ll == losses[w]
            assert np.array_equal(yy, y[w]) and np.array_equal(I.bf16_bits(X), Xb[w])
        before = loop.eng.x.copy()
        loop.eng.local_step(loop.g)                      # the engine steps on the shared-memory state
        np.testing.assert_allclose(loop.eng.x, before - 0.05 * loop.g, rtol=0, atol=1e-7)
    finally:
        loop.close()


def test_matching_decisions_finds_the_units_that_were_switched():
    """match_decisions reads switched ReLU decisions off the bias gradients.  Take the oracle's own gradient with
    three near-zero units deliberately switched (a stand-in for a device that decided them the other way) and give
    only its bias gradients as the hint: the same three units must come back, and the matched gradient must be that
    gradient exactly; with an unswitched hint nothing is matched."""
    dims = (64, 128, 128, 10)
    rng = np.random.default_rng(0)
    segs, P = I.mlp_segments(dims)
    off = {n: o for n, o, _ in segs}
    flat = np.zeros(P, np.float32)
    for name, o, shape in segs:
        n = int(np.prod(shape))
        flat[o:o + n] = rng.standard_normal(n).astype(np.float32) * (1 / np.sqrt(shape[-1]) if name[0] == "W" else 0.1)
    X = I.round_to_bf16(rng.standard_normal((128, 64)).astype(np.float32))
    y = rng.integers(0, 10, 128).astype(np.int32)
    # the units nearest to zero as they come (parameters and inputs are used as bf16 values, so a pre-activation
    # cannot be placed at will): two of layer 1 in different columns, one of layer 2
    _, g0, mid = MO.loss_and_grad(flat, X, y, dims, True, return_intermediates=True)
    o1 = np.dstack(np.unravel_index(np.argsort(np.abs(mid["z1"]), axis=None), mid["z1"].shape))[0]
    first = tuple(int(v) for v in o1[0])
    second = next(tuple(int(v) for v in bj) for bj in o1[1:] if bj[1] != first[1])
    third = tuple(int(v) for v in np.unravel_index(np.argmin(np.abs(mid["z2"])), mid["z2"].shape))
    want = sorted([(1,) + first, (1,) + second, (2,) + third])
    for layer, b, j in want:
        assert abs(mid["z%d" % layer][b, j]) < C.BAND_MAX
    _, g_sw = MO.loss_and_grad(flat, X, y, dims, True, flips=want)
    b1 = slice(off["b1"], off["b1"] + dims[1])
    b2 = slice(off["b2"], off["b2"] + dims[2])
    l0, gc, l1, gm, flips = C.match_decisions(flat, X, y, dims, g_sw[b1], g_sw[b2])
    assert sorted(tuple(f[:3]) for f in flips) == want
    np.testing.assert_array_equal(gm, g_sw)
    np.testing.assert_array_equal(gc, g0)
    assert np.abs(g_sw - g0).max() > 1e-4
    _, _, _, gm0, none = C.match_decisions(flat, X, y, dims, g0[b1], g0[b2])
    assert none == [] and np.array_equal(gm0, g0)
