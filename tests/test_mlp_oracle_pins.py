"""Pins of the MLP-gradient oracle (no GPU): finite differences, torch autograd, the textbook
softmax cross-entropy gradient, and the bfloat16 rounding rule."""
import numpy as np
import pytest

from oracle import mlp_oracle as MO
from paper_1906_12043_b200 import inputs as I

DIMS = (7, 6, 5, 4)


def tiny_problem(seed=0, M=9):
    rng = np.random.default_rng(seed)
    _, P = I.mlp_segments(DIMS)
    flat = rng.standard_normal(P) * 0.5
    X = rng.standard_normal((M, DIMS[0]))
    y = rng.integers(0, DIMS[3], M)
    return flat, X, y


def test_gradient_matches_central_finite_differences():
    flat, X, y = tiny_problem()
    _, g = MO.loss_and_grad(flat, X, y, DIMS, emulate_bf16=False)
    eps = 1e-6
    for i in range(len(flat)):
        a, b = flat.copy(), flat.copy()
        a[i] += eps
        b[i] -= eps
        fd = (MO.loss_and_grad(a, X, y, DIMS, False)[0] - MO.loss_and_grad(b, X, y, DIMS, False)[0]) / (2 * eps)
        assert abs(fd - g[i]) < 1e-6 + 1e-5 * abs(fd), (i, fd, g[i])


def test_gradient_and_loss_match_torch_autograd():
    torch = pytest.importorskip("torch")
    flat, X, y = tiny_problem(1, M=16)
    loss, g = MO.loss_and_grad(flat, X, y, DIMS, emulate_bf16=False)
    t = torch.tensor(flat, dtype=torch.float64, requires_grad=True)
    segs, _ = I.mlp_segments(DIMS)
    p = {n: t[o:o + int(np.prod(s))].reshape(s) for n, o, s in segs}
    h = torch.relu(torch.tensor(X) @ p["W1"].T + p["b1"])
    h = torch.relu(h @ p["W2"].T + p["b2"])
    z = h @ p["W3"].T + p["b3"]
    L = torch.nn.functional.cross_entropy(z, torch.tensor(y), reduction="mean")
    L.backward()
    assert abs(L.item() - loss) < 1e-12
    np.testing.assert_allclose(g, t.grad.numpy(), rtol=0, atol=1e-7)


def test_output_layer_gradient_is_softmax_minus_onehot_over_batch():
    flat, X, y = tiny_problem(2, M=5)
    _, g = MO.loss_and_grad(flat, X, y, DIMS, emulate_bf16=False)
    p = MO.split(flat, DIMS)
    h = np.maximum(np.maximum(X @ p["W1"].T + p["b1"], 0) @ p["W2"].T + p["b2"], 0)
    z = h @ p["W3"].T + p["b3"]
    sm = np.exp(z) / np.exp(z).sum(1, keepdims=True)
    sm[np.arange(5), y] -= 1
    segs, _ = I.mlp_segments(DIMS)
    off = dict((n, o) for n, o, _ in segs)
    np.testing.assert_allclose(g[off["b3"]:], sm.sum(0) / 5, atol=1e-7)
    np.testing.assert_allclose(g[off["W3"]:off["b3"]].reshape(DIMS[3], DIMS[2]), sm.T @ h / 5, atol=1e-7)


def test_loss_of_uniform_logits_is_log_classes_and_flat_layout_order():
    _, P = I.mlp_segments(DIMS)
    loss, g = MO.loss_and_grad(np.zeros(P), np.ones((3, DIMS[0])), np.array([0, 1, 2]), DIMS, False)
    assert abs(loss - np.log(DIMS[3])) < 1e-12
    segs, _ = I.mlp_segments(DIMS)
    assert [n for n, _, _ in segs] == ["W1", "b1", "W2", "b2", "W3", "b3"]
    off = dict((n, o) for n, o, _ in segs)
    assert np.all(g[:off["W3"]] == 0)              # dead network: only the last bias sees a gradient
    assert np.any(g[off["b3"]:] != 0)


def test_bf16_rounding_rule():
    f = lambda v: float(MO.bf16(np.array([v]))[0])
    assert f(1.0) == 1.0
    assert f(1.0 + 2 ** -8) == 1.0                 # tie -> even (mantissa ...0)
    assert f(1.0 + 3 * 2 ** -8) == 1.0 + 2 ** -6   # tie -> even (rounds up to ...10)
    assert f(1.0 + 2 ** -8 + 2 ** -20) == 1.0 + 2 ** -7
    assert f(-0.3) == -f(0.3)
    assert f(3.0e-3) != 3.0e-3 and abs(f(3.0e-3) - 3.0e-3) <= 3.0e-3 * 2 ** -8
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    a = (rng.standard_normal(100_000) * 10.0 ** rng.integers(-6, 6, 100_000)).astype(np.float32)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(MO.bf16(a).astype(np.float32), want)
    np.testing.assert_array_equal(I.round_to_bf16(a), want)
    np.testing.assert_array_equal(I.bf16_bits(want), torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def test_bf16_emulation_stays_close_to_exact_math():
    rng = np.random.default_rng(4)
    dims = (32, 24, 16, 10)
    _, P = I.mlp_segments(dims)
    flat = (rng.standard_normal(P) * 0.2).astype(np.float32)
    X = I.round_to_bf16(rng.standard_normal((64, 32)).astype(np.float32))
    y = rng.integers(0, 10, 64)
    l0, g0 = MO.loss_and_grad(flat, X, y, dims, False)
    l1, g1 = MO.loss_and_grad(flat, X, y, dims, True)
    assert abs(l0 - l1) < 2e-2 * abs(l0)
    assert np.abs(g0 - g1).max() < 3e-2 * np.abs(g0).max()
    assert np.any(g0 != g1)


def test_workload_recipe_shapes_and_labels():
    segs, P = I.mlp_segments()
    assert P == 1_863_690
    w = I.mlp_init_params(I.MLP_STUDENT_SEED)
    t = I.mlp_init_params(I.MLP_TEACHER_SEED)
    assert w.shape == (P,) and not np.array_equal(w, t)
    off = dict((n, (o, s)) for n, o, s in segs)
    assert np.all(w[off["b1"][0]:off["W2"][0]] == 0)
    assert abs(w[:802816].std() - 1 / np.sqrt(784)) < 2e-4
    X = I.mlp_batch(3, 5)
    assert X.shape == (128, 784) and np.array_equal(I.round_to_bf16(X), X)
    y = I.mlp_teacher_labels(X, t)
    assert y.shape == (128,) and y.min() >= 0 and y.max() <= 9 and len(set(y.tolist())) > 3


def test_a_flipped_relu_decision_is_the_gradient_of_the_network_with_that_gate_fixed():
    """`flips` takes a ReLU decision the other way.  Pin: with the gates g = (z > 0) treated as constants, the network
    is h = g * z, whose gradient torch's autograd gives for ANY gate pattern; for units whose pre-activation is (made)
    1e-9 away from zero, the oracle's flipped result must equal that gradient with the flipped gates, and the
    unflipped result the one with the original gates.  The intermediates it reports obey their definitions."""
    torch = pytest.importorskip("torch")
    flat, X, y = tiny_problem(5, M=12)
    segs, _ = I.mlp_segments(DIMS)
    off = dict((n, o) for n, o, _ in segs)
    # put z1[2][3] at -1e-9 and z2[7][1] at +1e-9 by moving the two biases (other samples keep ordinary values)
    _, _, mid = MO.loss_and_grad(flat, X, y, DIMS, False, return_intermediates=True)
    flat[off["b1"] + 3] -= mid["z1"][2, 3] + 1e-9
    _, _, mid = MO.loss_and_grad(flat, X, y, DIMS, False, return_intermediates=True)
    flat[off["b2"] + 1] -= mid["z2"][7, 1] - 1e-9
    loss0, g0, mid = MO.loss_and_grad(flat, X, y, DIMS, False, return_intermediates=True)
    assert abs(mid["z1"][2, 3] + 1e-9) < 1e-12 and abs(mid["z2"][7, 1] - 1e-9) < 1e-12
    assert not mid["on1"][2, 3] and mid["on2"][7, 1]
    flips = [(1, 2, 3), (2, 7, 1)]
    loss1, g1, mid1 = MO.loss_and_grad(flat, X, y, DIMS, False, flips=flips, return_intermediates=True)
    assert mid1["on1"][2, 3] and not mid1["on2"][7, 1] and mid1["h2"][7, 1] == 0
    assert (mid1["on1"] != mid["on1"]).sum() == 1 and (mid1["on2"] != mid["on2"]).sum() == 1

    def gated(on1, on2):
        t = torch.tensor(flat, dtype=torch.float64, requires_grad=True)
        p = {n: t[o:o + int(np.prod(s))].reshape(s) for n, o, s in segs}
        h = (torch.tensor(X) @ p["W1"].T + p["b1"]) * torch.tensor(on1, dtype=torch.float64)
        h = (h @ p["W2"].T + p["b2"]) * torch.tensor(on2, dtype=torch.float64)
        L = torch.nn.functional.cross_entropy(h @ p["W3"].T + p["b3"], torch.tensor(y), reduction="mean")
        L.backward()
        return L.item(), t.grad.numpy()

    for (loss, g, m) in ((loss0, g0, mid), (loss1, g1, mid1)):
        want_l, want_g = gated(m["on1"], m["on2"])
        assert abs(want_l - loss) < 1e-8
        np.testing.assert_allclose(g, want_g, rtol=0, atol=1e-7)
    assert np.abs(g1 - g0).max() > 1e-4                  # the flip matters: one sample's term switched
    # definitions of the reported intermediates
    p = MO.split(flat, DIMS)
    np.testing.assert_allclose(mid["pre2"], mid["dz3"] @ p["W3"], atol=1e-15)
    np.testing.assert_allclose(mid["dz2"], mid["pre2"] * mid["on2"], atol=0)
    np.testing.assert_allclose(mid["pre1"], mid["dz2"] @ p["W2"], atol=1e-15)
    np.testing.assert_allclose(mid["dz1"], mid["pre1"] * mid["on1"], atol=0)
    np.testing.assert_allclose(g0[off["b2"]:off["W3"]], mid["dz2"].sum(0), atol=1e-7)
    np.testing.assert_allclose(g0[off["b1"]:off["W2"]], mid["dz1"].sum(0), atol=1e-7)
