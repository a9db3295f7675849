"""Pins that tie the CPU oracle to something other than itself (no GPU needed).

Each test checks the oracle against what Algorithm 1 of the paper and plain algebra fix:
hand-computed rounds (tests/golden), the closed forms from the proof of Lemma 2
(eqs. "local_represent" / "average_represent"), invariants of line 6 (the merge), special
cases that reduce to single-worker momentum SGD or to plain model averaging, and an
exact-rational brute force written here straight from Algorithm 1.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle.cocod_oracle import OracleEngine

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MODES = ["ref", "f64", "mirror"]


# ----------------------------------------------------------------------------- helpers
def load_fixture(name):
    fx = {"grad": {}, "expect_x": {}, "expect_v": {}, "expect_mean": {}, "batch_sizes": None}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            key, vals = line[0], line[1:]
            if key in ("K", "P", "k", "rounds"):
                fx[key] = int(vals[0])
            elif key in ("lr", "mu", "wd"):
                fx[key] = float(vals[0])
            elif key == "x0":
                fx["x0"] = np.array(vals, float)
            elif key == "batch_sizes":
                fx["batch_sizes"] = np.array(vals, float)
            elif key == "grad":
                fx["grad"][(int(vals[0]), int(vals[1]))] = np.array(vals[2:], float)
            elif key == "expect_x":
                fx["expect_x"][(int(vals[0]), int(vals[1]))] = np.array(vals[2:], float)
            elif key == "expect_v":
                fx["expect_v"][int(vals[0])] = np.array(vals[1:], float)
            elif key == "expect_mean":
                fx["expect_mean"][int(vals[0])] = np.array(vals[1:], float)
            else:
                raise ValueError(key)
    return fx


def rand_grads(rng, K, P, steps, scale=0.01):
    return rng.standard_normal((steps, K, P)) * scale


def run_oracle(mode, K, P, lr, mu, wd, k, rounds, x0, G, M=None):
    eng = OracleEngine(K, P, lr, mu, wd, mode=mode, batch_sizes=M)
    eng.set_params(x0)
    eng.run(lambda t: G[t], k, rounds)
    return eng


def tol(mode):
    return 1e-12 if mode == "f64" else 2e-5


# ----------------------------------------------------------------------------- P10: hand-computed rounds
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", ["algorithm1_k2_p8.txt", "algorithm1_weight_decay_k1.txt",
                                  "algorithm1_weighted_mean.txt"])
def test_golden_hand_computed_rounds(name, mode):
    fx = load_fixture(name)
    K, P, k = fx["K"], fx["P"], fx["k"]
    eng = OracleEngine(K, P, fx["lr"], fx["mu"], fx["wd"], mode=mode, batch_sizes=fx["batch_sizes"])
    eng.set_params(fx["x0"])
    for r in range(fx["rounds"]):
        eng.comm_begin()
        np.testing.assert_array_equal(eng.mean.astype(float), fx["expect_mean"][r])
        for s in range(k):
            g = np.stack([fx["grad"][(r * k + s, w)] for w in range(K)])
            eng.local_step(g)
        eng.comm_end()
        for w in range(K):
            np.testing.assert_array_equal(eng.x[w].astype(float), fx["expect_x"][(r, w)],
                                          err_msg=f"round {r} worker {w}")
    for w in range(K):
        np.testing.assert_array_equal(eng.v[w].astype(float), fx["expect_v"][w])


# ----------------------------------------------------------------------------- P11: exact-rational brute force
def algorithm1_exact(K, P, lr, mu, wd, k, rounds, x0, G, M=None):
    """Algorithm 1 in exact rational arithmetic, scalar loops, written from the paper."""
    x = [[Fraction(x0[p]) for p in range(P)] for _ in range(K)]
    v = [[Fraction(0)] * P for _ in range(K)]
    w = [Fraction(1, K)] * K if M is None else [Fraction(m) / sum(Fraction(mm) for mm in M) for m in M]
    lr, mu, wd = Fraction(lr), Fraction(mu), Fraction(wd)
    for r in range(rounds):
        stored = [row[:] for row in x]                                        # Step I: store x_t^i
        xhat = [sum(w[i] * stored[i][p] for i in range(K)) for p in range(P)]  # weighted mean
        for s in range(k):                                                   # Step II
            t = r * k + s
            for i in range(K):
                for p in range(P):
                    d = Fraction(G[t][i][p]) + wd * x[i][p]
                    v[i][p] = mu * v[i][p] + d
                    x[i][p] = x[i][p] - lr * v[i][p]
        for i in range(K):                                                   # line 6
            for p in range(P):
                x[i][p] = xhat[p] + (x[i][p] - stored[i][p])
    return x, v


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("seed", range(6))
def test_brute_force_exact_rational_dyadic(seed, mode):
    """Dyadic inputs and hyper-parameters keep every value exact in fp32 for a few steps, so
    all three modes must agree with exact rational arithmetic bit for bit."""
    rng = np.random.default_rng(seed)
    K = int(rng.choice([1, 2, 3, 4]))
    P = int(rng.integers(1, 6))
    k = int(rng.integers(1, 3))
    rounds = 2
    lr, mu, wd = 0.5, float(rng.choice([0.0, 0.5])), float(rng.choice([0.0, 0.25]))
    x0 = rng.integers(-4, 5, P).astype(float) / 2
    G = rng.integers(-4, 5, (k * rounds, K, P)).astype(float)
    M = None
    if K in (2, 4) and seed % 2:
        M = [1, 3] if K == 2 else [1, 1, 2, 4]            # weights stay dyadic
    ex, ev = algorithm1_exact(K, P, lr, mu, wd, k, rounds, x0, G, M)
    eng = run_oracle(mode, K, P, lr, mu, wd, k, rounds, x0, G, M)
    want_x = np.array([[float(c) for c in row] for row in ex])
    want_v = np.array([[float(c) for c in row] for row in ev])
    if K == 3:      # 1/3 is not dyadic: exact up to rounding only
        np.testing.assert_allclose(eng.x, want_x, rtol=0, atol=1e-5)
        np.testing.assert_allclose(eng.v, want_v, rtol=0, atol=1e-5)
    else:
        np.testing.assert_array_equal(eng.x.astype(float), want_x)
        np.testing.assert_array_equal(eng.v.astype(float), want_v)


def algorithm1_numpy(K, P, lr, mu, wd, k, rounds, x0, G, M=None):
    """Second, vectorised fp64 restatement of Algorithm 1 (independent of the C code)."""
    x = np.tile(np.asarray(x0, float), (K, 1))
    v = np.zeros((K, P))
    w = np.full(K, 1.0 / K) if M is None else np.asarray(M, float) / np.sum(M)
    for r in range(rounds):
        stored = x.copy()
        xhat = w @ stored
        for s in range(k):
            v = mu * v + (G[r * k + s] + wd * x)
            x = x - lr * v
        x = xhat[None, :] + (x - stored)
    return x, v


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("seed", range(8))
def test_random_cases_against_numpy_restatement(seed, mode):
    rng = np.random.default_rng(100 + seed)
    K, P = int(rng.integers(1, 6)), int(rng.integers(1, 65))
    k, rounds = int(rng.integers(1, 5)), int(rng.integers(1, 5))
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = rand_grads(rng, K, P, k * rounds).astype(np.float32)
    M = rng.integers(1, 5, K).astype(float) if seed % 2 else None
    wx, wv = algorithm1_numpy(K, P, float(lr), float(mu), float(wd), k, rounds, x0, G.astype(float), M)
    eng = run_oracle(mode, K, P, lr, mu, wd, k, rounds, x0, G, M)
    np.testing.assert_allclose(eng.x, wx, rtol=0, atol=tol(mode) * 0.05)
    np.testing.assert_allclose(eng.v, wv, rtol=0, atol=tol(mode) * 0.05)


# ----------------------------------------------------------------------------- P1 / P7: reductions to single-worker SGD
def momentum_sgd_single(lr, mu, wd, x0, g_seq):
    """Textbook single-worker momentum SGD with coupled weight decay (PyTorch SGD form)."""
    x, v = np.asarray(x0, float).copy(), np.zeros(len(x0))
    for g in g_seq:
        v = mu * v + g + wd * x
        x = x - lr * v
    return x, v


@pytest.mark.parametrize("mode", MODES)
def test_K1_merge_is_identity_and_run_is_single_worker_sgd(mode):
    rng = np.random.default_rng(1)
    P, k, rounds = 37, 3, 4
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = rand_grads(rng, 1, P, k * rounds).astype(np.float32)
    eng = OracleEngine(1, P, lr, mu, wd, mode=mode)
    eng.set_params(x0)
    for r in range(rounds):
        eng.comm_begin()
        for s in range(k):
            eng.local_step(G[r * k + s])
        before = eng.x.copy()
        eng.comm_end()
        if mode == "ref":      # fp32 operands, fp64 evaluation: every intermediate is exact
            np.testing.assert_array_equal(eng.x, before)
        else:                  # "snap + (x - snap)" may move x by one rounding of the drift
            np.testing.assert_allclose(eng.x, before, rtol=0, atol=1e-8 if mode == "mirror" else 1e-16)
    wx, wv = momentum_sgd_single(float(lr), float(mu), float(wd), x0, G[:, 0].astype(float))
    np.testing.assert_allclose(eng.x[0], wx, rtol=0, atol=tol(mode) * 0.05)
    np.testing.assert_allclose(eng.v[0], wv, rtol=0, atol=tol(mode) * 0.05)


@pytest.mark.parametrize("mode", MODES)
def test_identical_gradients_keep_replicas_identical(mode):
    rng = np.random.default_rng(2)
    K, P, k, rounds = 4, 19, 2, 3
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    g1 = rand_grads(rng, 1, P, k * rounds).astype(np.float32)
    G = np.repeat(g1, K, axis=1)
    eng = run_oracle(mode, K, P, lr, mu, wd, k, rounds, x0, G)
    for i in range(1, K):
        np.testing.assert_array_equal(eng.x[i], eng.x[0])
    wx, _ = momentum_sgd_single(float(lr), float(mu), float(wd), x0, g1[:, 0].astype(float))
    np.testing.assert_allclose(eng.x[0], wx, rtol=0, atol=tol(mode) * 0.05)


# ----------------------------------------------------------------------------- P2: zero drift = plain model averaging
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("weighted", [False, True])
def test_zero_drift_merge_is_plain_model_averaging(mode, weighted):
    rng = np.random.default_rng(3)
    K, P = 5, 23
    X = (rng.standard_normal((K, P)) * 0.1).astype(np.float32)
    M = np.array([1.0, 2.0, 3.0, 2.0, 8.0]) if weighted else None
    eng = OracleEngine(K, P, 0.1, 0.9, 0.0, mode=mode, batch_sizes=M)
    eng.set_params_all(X)
    eng.comm_begin()
    eng.comm_end()
    w = np.full(K, 1 / K) if M is None else M / M.sum()
    want = w @ X.astype(float)
    for i in range(K):
        np.testing.assert_array_equal(eng.x[i], eng.mean)          # m + 0 = m exactly
        np.testing.assert_allclose(eng.x[i], want, rtol=0, atol=1e-15 if mode == "f64" else 3e-8)


# ----------------------------------------------------------------------------- P3 / P6: merge invariants
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("weighted", [False, True])
def test_merge_preserves_the_weighted_mean_and_subtracts_old_drift(mode, weighted):
    rng = np.random.default_rng(4)
    K, P, k = 6, 41, 3
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    M = rng.integers(1, 9, K).astype(float) if weighted else None
    w = np.full(K, 1 / K) if M is None else M / M.sum()
    eng = OracleEngine(K, P, lr, mu, wd, mode=mode, batch_sizes=M)
    eng.set_params_all((rng.standard_normal((K, P)) * 0.05).astype(np.float32))
    for r in range(3):
        eng.comm_begin()
        x_t = eng.x.astype(float).copy()
        for s in range(k):
            eng.local_step((rng.standard_normal((K, P)) * 0.01).astype(np.float32))
        pre = eng.x.astype(float).copy()
        eng.comm_end()
        post = eng.x.astype(float)
        a = 1e-13 if mode == "f64" else 5e-8
        # mean_i x_i unchanged by line 6
        np.testing.assert_allclose(w @ post, w @ pre, rtol=0, atol=a)
        # e_i := x_i - xbar obeys e_i(after) = e_i(t+k) - e_i(t)
        e = lambda X: X - (w @ X)[None, :]
        np.testing.assert_allclose(e(post), e(pre) - e(x_t), rtol=0, atol=a)


# ----------------------------------------------------------------------------- P8: first merge is an identity
@pytest.mark.parametrize("mode", MODES)
def test_first_merge_is_identity_because_all_workers_start_equal(mode):
    rng = np.random.default_rng(5)
    K, P, k = 4, 33, 4
    eng = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode=mode)
    eng.set_params((rng.standard_normal(P) * 0.01).astype(np.float32))
    eng.comm_begin()
    np.testing.assert_array_equal(eng.mean, eng.x[0])       # mean of equal values (K = 4: exact)
    for s in range(k):
        eng.local_step((rng.standard_normal((K, P)) * 0.01).astype(np.float32))
    pre = eng.x.copy()
    eng.comm_end()
    np.testing.assert_allclose(eng.x, pre, rtol=0, atol={"ref": 0, "mirror": 1e-8, "f64": 1e-16}[mode])


# ----------------------------------------------------------------------------- P4: closed forms of the proof (plain SGD)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("weighted", [False, True])
def test_closed_form_local_and_average_representation(mode, weighted):
    """mu = wd = 0.  With t' = (floor(t/k) - 1) k (clamped at 0):
         x_t^i   = xhat_{t'} - gamma sum_{tau=t'}^{t-1} G_tau^i                  (local_represent)
         xhat_t' = x0 - gamma sum_{tau<t'} sum_j w_j G_tau^j                      (average_represent, unrolled)
       evaluated directly from the gradient stream, no simulation."""
    rng = np.random.default_rng(6)
    K, P, k, rounds = 4, 29, 3, 4
    lr = np.float32(0.125)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = rand_grads(rng, K, P, k * rounds).astype(np.float32)
    M = np.array([1.0, 2.0, 2.0, 3.0]) if weighted else None
    w = np.full(K, 1 / K) if M is None else M / M.sum()
    Gd = G.astype(float)
    gbar = np.einsum("j,tjp->tp", w, Gd)

    def closed(t):
        tp = max(0, (t // k - 1) * k)
        xhat = x0.astype(float) - float(lr) * gbar[:tp].sum(0)
        return xhat[None, :] - float(lr) * Gd[tp:t].sum(0)

    eng = OracleEngine(K, P, lr, 0.0, 0.0, mode=mode, batch_sizes=M)
    eng.set_params(x0)
    t = 0
    for r in range(rounds):
        eng.comm_begin()
        for s in range(k):
            eng.local_step(G[t])
            t += 1
            if s < k - 1:      # mid-round: the in-memory model is the represented x_t^i
                np.testing.assert_allclose(eng.x, closed(t), rtol=0, atol=tol(mode) * 0.02)
        eng.comm_end()
        np.testing.assert_allclose(eng.x, closed(t), rtol=0, atol=tol(mode) * 0.02)


# ----------------------------------------------------------------------------- P5: the mean obeys single-worker momentum SGD
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("weighted", [False, True])
def test_worker_mean_follows_single_worker_recursion(mode, weighted):
    """The update is linear in (x, v) and the synthetic gradients do not depend on x, so
    (xbar, vbar) = weighted means over workers follow momentum SGD driven by gbar, and
    line 6 leaves xbar untouched: a K-free recursion predicts mean_i x_i after any run."""
    rng = np.random.default_rng(7)
    K, P, k, rounds = 8, 31, 4, 5
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = rand_grads(rng, K, P, k * rounds).astype(np.float32)
    M = rng.integers(1, 5, K).astype(float) if weighted else None
    w = np.full(K, 1 / K) if M is None else M / M.sum()
    gbar = np.einsum("j,tjp->tp", w, G.astype(float))
    wx, wv = momentum_sgd_single(float(lr), float(mu), float(wd), x0, gbar)
    eng = run_oracle(mode, K, P, lr, mu, wd, k, rounds, x0, G, M)
    np.testing.assert_allclose(w @ eng.x.astype(float), wx, rtol=0, atol=tol(mode) * 0.05)
    np.testing.assert_allclose(w @ eng.v.astype(float), wv, rtol=0, atol=tol(mode) * 0.05)


# ----------------------------------------------------------------------------- P9: k = 1
@pytest.mark.parametrize("mode", MODES)
def test_period_one_each_worker_steps_from_the_average(mode):
    rng = np.random.default_rng(8)
    K, P = 3, 17
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    eng = OracleEngine(K, P, lr, mu, wd, mode=mode)
    eng.set_params_all((rng.standard_normal((K, P)) * 0.05).astype(np.float32))
    for r in range(4):
        eng.comm_begin()
        xhat = eng.mean.astype(float).copy()
        eng.local_step((rng.standard_normal((K, P)) * 0.01).astype(np.float32))
        eng.comm_end()
        want = xhat[None, :] - float(lr) * eng.v.astype(float)
        np.testing.assert_allclose(eng.x, want, rtol=0, atol=1e-14 if mode == "f64" else 3e-8)


# ----------------------------------------------------------------------------- mode relations and index sanity
def test_mirror_uses_fused_multiply_add_and_ref_rounds_once():
    """A value where fused and unfused fp32 evaluation differ pins which one 'mirror' is."""
    x = np.float32(1.0 + 2.0 ** -12)
    lr = np.float32(1.0 + 2.0 ** -12)
    g = np.float32(-1.0)                      # v = g = -1 ; x_new = x + lr (mu = 0, wd = 0)
    eng = OracleEngine(1, 1, lr, 0.0, 0.0, mode="mirror")
    eng.set_params([x])
    eng.local_step(np.array([[g]], np.float32))
    assert eng.x[0, 0] == np.float32(float(x) + float(lr))
    # weight decay term: d = fma(wd, x, g) keeps the exact product before adding g
    wd = np.float32(1.0 + 2.0 ** -12)
    eng = OracleEngine(1, 1, 0.0, 0.0, wd, mode="mirror")
    eng.set_params([x])
    eng.local_step(np.array([[np.float32(-1.0)]], np.float32))
    exact = float(wd) * float(x) - 1.0                      # 2^-11 + 2^-24: needs the unrounded product
    assert eng.v[0, 0] == np.float32(exact)
    assert np.float32(np.float32(wd * x) + np.float32(-1.0)) != np.float32(exact)


def test_modes_agree_to_rounding_on_workload_shaped_input():
    rng = np.random.default_rng(9)
    K, P, k, rounds = 4, 1000, 4, 10
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = rand_grads(rng, K, P, k * rounds).astype(np.float32)
    e = {m: run_oracle(m, K, P, lr, mu, wd, k, rounds, x0, G) for m in MODES}
    scale = np.sqrt(np.mean(e["f64"].x ** 2))
    for m in ("ref", "mirror"):
        err = np.abs(e[m].x - e["f64"].x).max() / scale
        assert err < 1e-5, (m, err)
    # and the modes are not accidentally the same code path
    assert np.any(e["ref"].x != e["mirror"].x)


def test_rows_are_workers_and_columns_are_parameters():
    """A transposed or mis-strided access would mix these distinct per-row, per-column values."""
    K, P = 3, 5
    X = (np.arange(K)[:, None] * 100.0 + np.arange(P)[None, :]).astype(np.float32)
    eng = OracleEngine(K, P, 1.0, 0.0, 0.0, mode="ref")
    eng.set_params_all(X)
    eng.comm_begin()
    np.testing.assert_array_equal(eng.mean, 100.0 + np.arange(P))
    g = np.zeros((K, P), np.float32)
    g[1, 2] = 7.0
    eng.local_step(g)
    eng.comm_end()
    want = np.tile(100.0 + np.arange(P), (K, 1))
    want[1, 2] -= 7.0
    np.testing.assert_array_equal(eng.x, want)


def test_state_machine_rejects_double_begin_and_end_without_begin():
    eng = OracleEngine(2, 2, 0.1, 0.0, 0.0)
    with pytest.raises(RuntimeError):
        eng.comm_end()
    eng.comm_begin()
    with pytest.raises(RuntimeError):
        eng.comm_begin()


# ----------------------------------------------------------------------------- the sequential schemes
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("weighted", [False, True])
def test_ssgd_equals_one_worker_on_the_averaged_gradient(mode, weighted):
    """S-SGD with K workers is single-worker momentum SGD driven by the weighted mean gradient (more
    workers = a larger mini-batch); all replicas stay identical."""
    rng = np.random.default_rng(21)
    K, P, steps = 5, 27, 7
    lr, mu, wd = np.float32(0.1), np.float32(0.9), np.float32(5e-4)
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = rand_grads(rng, K, P, steps).astype(np.float32)
    M = rng.integers(1, 6, K).astype(float) if weighted else None
    w = np.full(K, 1 / K) if M is None else M / M.sum()
    eng = OracleEngine(K, P, lr, mu, wd, mode=mode, batch_sizes=M)
    eng.set_params(x0)
    for t in range(steps):
        eng.ssgd_step(G[t])
    for i in range(1, K):
        np.testing.assert_array_equal(eng.x[i], eng.x[0])
    wx, wv = momentum_sgd_single(float(lr), float(mu), float(wd), x0, np.einsum("j,tjp->tp", w, G.astype(float)))
    np.testing.assert_allclose(eng.x[0], wx, rtol=0, atol=tol(mode) * 0.05)
    np.testing.assert_allclose(eng.v[0], wv, rtol=0, atol=tol(mode) * 0.05)


@pytest.mark.parametrize("mode", MODES)
def test_local_sgd_average_is_the_zero_drift_merge(mode):
    """Local-SGD's averaging step equals Step I + line 6 of Algorithm 1 with no local step in between,
    and with k = 1 and plain SGD, Local-SGD and S-SGD produce the same models."""
    rng = np.random.default_rng(22)
    K, P = 4, 19
    X = (rng.standard_normal((K, P)) * 0.1).astype(np.float32)
    a = OracleEngine(K, P, 0.1, 0.0, 0.0, mode=mode)
    b = OracleEngine(K, P, 0.1, 0.0, 0.0, mode=mode)
    a.set_params_all(X)
    b.set_params_all(X)
    a.local_sgd_average()
    b.comm_begin()
    b.comm_end()
    np.testing.assert_array_equal(a.x, b.x)
    # k = 1, mu = wd = 0: average(x - lr g_i) = x - lr * mean(g)
    g = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
    c = OracleEngine(K, P, 0.1, 0.0, 0.0, mode=mode)
    c.set_params_all(a.x)
    a.local_step(g)
    a.local_sgd_average()
    c.ssgd_step(g)
    np.testing.assert_allclose(a.x, c.x, rtol=0, atol=1e-15 if mode == "f64" else 5e-8)


# ----------------------------------------------------------------------------- Step I's mean over many workers
# The fp32 "mirror" sums the workers in blocks of 8 rows (pairwise tree inside a block, block sums accumulated in
# order, a ragged last block); the cases below hold that path -- and the plain loops of the other two modes -- to
# exact rational arithmetic and to an error bound, at worker counts with 2 to 125 blocks and every kind of tail.
MANY_K = [9, 15, 16, 17, 64, 1000]


def exact_weighted_mean(X, M=None):
    """Step I's x_hat = sum_i (M_i / sum_j M_j) x^i in exact rational arithmetic (scalar loops)."""
    K, P = X.shape
    tot = Fraction(K) if M is None else sum(Fraction(float(m)) for m in M)
    w = [Fraction(1) / tot if M is None else Fraction(float(M[i])) / tot for i in range(K)]
    return [sum(w[i] * Fraction(float(X[i, p])) for i in range(K)) for p in range(P)]


def mean_of(mode, X, M=None):
    K, P = X.shape
    eng = OracleEngine(K, P, 0.1, 0.0, 0.0, mode=mode, batch_sizes=M)
    eng.set_params_all(X)
    eng.comm_begin()
    return eng


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("K", MANY_K)
def test_many_worker_mean_is_exact_on_dyadic_inputs(K, mode):
    """Small dyadic rows: every partial sum is exact in fp32 in any order, so the only roundings left are 1/K and
    the final product (none at all when K is a power of two)."""
    rng = np.random.default_rng(K)
    P = 11
    X = (rng.integers(-64, 65, (K, P)) / 16).astype(np.float32)
    eng = mean_of(mode, X)
    want = np.array([float(c) for c in exact_weighted_mean(X)])
    if K & (K - 1) == 0:
        np.testing.assert_array_equal(eng.mean.astype(np.float64), want)
    else:
        bound = 2.0 ** -23 * np.abs(want) if mode != "f64" else 2.0 ** -52 * np.abs(want)
        assert np.all(np.abs(eng.mean.astype(np.float64) - want) <= bound)
    # line 6 with zero drift then hands exactly that mean to every worker
    eng.comm_end()
    for i in range(K):
        np.testing.assert_array_equal(eng.x[i], eng.mean)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("K", MANY_K)
def test_many_worker_mean_counts_every_worker_exactly_once(K, mode):
    """Worker i is the only one with a non-zero entry in column i: a dropped, doubled or misplaced row (or whole
    block of rows) changes that column from 2^j / K to 0 or to a multiple of it."""
    X = np.zeros((K, K), np.float32)
    vals = 2.0 ** (np.arange(K) % 7 - 3)
    X[np.arange(K), np.arange(K)] = vals
    eng = mean_of(mode, X)
    want = vals / K
    np.testing.assert_allclose(eng.mean.astype(np.float64), want, rtol=2.0 ** -22, atol=0)
    # unequal batch sizes that are powers of two with a power-of-two total keep the weights dyadic: exact
    if K == 16:
        M = np.array([8] + [1] * 8 + [2] * 4 + [4] * 2 + [32], float)          # sums to 64
        eng = mean_of(mode, X, M)
        np.testing.assert_array_equal(eng.mean.astype(np.float64), vals * M / 64.0)


@pytest.mark.parametrize("weighted", [False, True])
@pytest.mark.parametrize("K", MANY_K)
def test_many_worker_mean_within_its_rounding_bound_on_gaussian_inputs(K, weighted):
    """fp32 mirror against exact arithmetic on workload-shaped values: the tree-of-8 order performs at most
    3 + K/8 dependent additions per column, plus one rounding of each weight and of each product (weighted) or of
    1/K and the final product (equal sizes).  The fp64-evaluated modes must sit within one fp32 rounding."""
    rng = np.random.default_rng(100 + K)
    P = 64
    X = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
    M = rng.integers(1, 9, K).astype(float) if weighted else None
    exact = exact_weighted_mean(X, M)
    want = np.array([float(c) for c in exact])
    w = np.full(K, 1.0 / K) if M is None else M / M.sum()
    mass = np.abs(w[:, None] * X.astype(np.float64)).sum(axis=0)              # sum_i |w_i x_i| per column
    mir = mean_of("mirror", X, M).mean.astype(np.float64)
    assert np.all(np.abs(mir - want) <= (5 + K / 8) * 2.0 ** -24 * mass)
    ref = mean_of("ref", X, M).mean.astype(np.float64)
    assert np.all(np.abs(ref - want) <= 2.0 ** -24 * np.abs(want) + 1e-16 * mass)
    f64 = mean_of("f64", X.astype(np.float64), M).mean
    assert np.all(np.abs(f64 - want) <= 1e-15 * mass)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("K", [9, 17, 64])
def test_sequential_schemes_with_many_workers(K, mode):
    """Local-SGD's averaging and S-SGD's gradient averaging use the same mean: at worker counts that span
    several blocks they must give every worker the exact weighted mean (dyadic inputs, to the rounding of 1/K)."""
    rng = np.random.default_rng(K + 7)
    P = 13
    X = (rng.integers(-32, 33, (K, P)) / 8).astype(np.float32)
    want = np.array([float(c) for c in exact_weighted_mean(X)])
    tol_k = 0.0 if K & (K - 1) == 0 else 2.0 ** -23
    a = OracleEngine(K, P, 0.5, 0.0, 0.0, mode=mode)
    a.set_params_all(X)
    a.local_sgd_average()
    for i in range(K):
        assert np.all(np.abs(a.x[i].astype(np.float64) - want) <= tol_k * np.abs(want))
    # S-SGD from x = 0 with lr = 1/2, mu = wd = 0: x = -mean(g) / 2 on every worker
    b = OracleEngine(K, P, 0.5, 0.0, 0.0, mode=mode)
    b.ssgd_step(X)
    for i in range(K):
        assert np.all(np.abs(b.x[i].astype(np.float64) + want / 2) <= tol_k * np.abs(want) / 2)
