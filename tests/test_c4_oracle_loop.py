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
        losses, Xb, y = loop.gradients(tau)
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
