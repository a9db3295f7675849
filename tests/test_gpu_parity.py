"""GPU parity: the CUDA engine, called through the C boundary, against the CPU oracle on the
same seeded inputs.

Bars (fp32 path):
  * against the oracle's "ref" mode (fp32-stored, fp64-evaluated): per element
        |gpu - ref| <= rtol * max(|ref|, rms(ref))
    with rtol 1e-6 after one round and 1e-5 after a full run, on x and on the momentum v;
  * against the oracle's "mirror" mode (same fp32 operation order): bit for bit.
"""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle.cocod_oracle import OracleEngine
from paper_1906_12043_b200 import inputs as I

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def E():
    from paper_1906_12043_b200 import build, engine
    build.build()
    engine.load()
    return engine


def assert_close_scaled(got, ref, rtol, what=""):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    scale = np.maximum(np.abs(ref), np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref) / np.maximum(scale, 1e-300)
    worst = float(err.max()) if err.size else 0.0
    assert worst <= rtol, f"{what}: max scaled error {worst:.3e} > {rtol:.1e}"
    return worst


def assert_bit_equal(got, ref, what=""):
    got = np.ascontiguousarray(got, np.float32).view(np.uint32)
    ref = np.ascontiguousarray(ref, np.float32).view(np.uint32)
    bad = np.nonzero(got != ref)
    assert bad[0].size == 0, f"{what}: {bad[0].size} elements differ, first at {[b[0] for b in bad]}"


def cpu(t):
    return t.detach().cpu().numpy()


def run_both(E, K, P, lr, mu, wd, k, rounds, x0, grad_fn, M=None, snapshot=None, side="own",
             check_round=None):
    """Drive the engine and both oracle modes with the same bytes; returns (eng, ref, mirror)."""
    eng = E.Engine(K, P, lr, mu, wd)
    if snapshot is not None:
        eng.set_option(E.OPT_SNAPSHOT, snapshot)
    if M is not None:
        eng.set_batch_sizes(M)
    eng.set_params(torch.from_numpy(x0).cuda())
    side_stream = {"own": torch.cuda.Stream(), "same": None,
                   "high": torch.cuda.Stream(priority=-1)}[side]
    ref = OracleEngine(K, P, lr, mu, wd, mode="ref", batch_sizes=M)
    mir = OracleEngine(K, P, lr, mu, wd, mode="mirror", batch_sizes=M)
    ref.set_params(x0)
    mir.set_params(x0)
    keep = []
    for r in range(rounds):
        eng.comm_begin(side_stream if side_stream is not None else torch.cuda.current_stream())
        ref.comm_begin()
        mir.comm_begin()
        for s in range(k):
            g = np.ascontiguousarray(grad_fn(r * k + s), np.float32)
            gd = torch.from_numpy(g).cuda()
            keep.append(gd)
            eng.local_step(gd)
            ref.local_step(g)
            mir.local_step(g)
        eng.comm_end()
        ref.comm_end()
        mir.comm_end()
        if check_round is not None:
            check_round(r, eng, ref, mir)
    eng.sync()
    return eng, ref, mir


# ----------------------------------------------------------------------------- inputs: device == host
def test_device_generator_matches_host_bits(E):
    n = 200_003
    for (seed, stream, w, t, p0, sigma) in [(0, I.STREAM_X0, 0, 0, 0, 0.01), (1234, I.STREAM_GRAD, 5, 17, 0, 0.01),
                                            (1234, I.STREAM_GRAD, 15, 99, 2 ** 33 + 5, 1.0)]:
        out = torch.empty(n, dtype=torch.float32, device="cuda")
        I.device_gaussian_into(out, seed, stream, w, t, p0, sigma)
        assert_bit_equal(cpu(out), I.gaussian(seed, stream, w, t, p0, n, sigma), f"stream {stream}")
    g = torch.empty((3, 1001), dtype=torch.float32, device="cuda")
    I.device_gradients_into(g, step=4)
    assert_bit_equal(cpu(g), I.gradients(3, 1001, 4))


# ----------------------------------------------------------------------------- hand-computed rounds
@pytest.mark.parametrize("snapshot", [0, 1])
@pytest.mark.parametrize("name", ["algorithm1_k2_p8.txt", "algorithm1_weight_decay_k1.txt",
                                  "algorithm1_weighted_mean.txt"])
def test_golden_rounds_through_the_c_boundary(E, name, snapshot):
    from test_oracle_pins import load_fixture
    fx = load_fixture(name)
    K, P, k = fx["K"], fx["P"], fx["k"]
    eng = E.Engine(K, P, fx["lr"], fx["mu"], fx["wd"])
    eng.set_option(E.OPT_SNAPSHOT, snapshot)
    if fx["batch_sizes"] is not None:
        eng.set_batch_sizes(fx["batch_sizes"])
    eng.set_params(fx["x0"].astype(np.float32))
    side = torch.cuda.Stream()
    for r in range(fx["rounds"]):
        eng.comm_begin(side)
        np.testing.assert_array_equal(cpu(eng.get_mean()).astype(float), fx["expect_mean"][r])
        for s in range(k):
            g = np.stack([fx["grad"][(r * k + s, w)] for w in range(K)]).astype(np.float32)
            eng.local_step(torch.from_numpy(g).cuda())
        eng.comm_end()
        x = cpu(eng.get_params()).astype(float)
        for w in range(K):
            np.testing.assert_array_equal(x[w], fx["expect_x"][(r, w)])
    v = cpu(eng.get_momentum()).astype(float)
    for w in range(K):
        np.testing.assert_array_equal(v[w], fx["expect_v"][w])
    assert eng.step_count == k * fx["rounds"]


# ----------------------------------------------------------------------------- config 1, element by element
@pytest.mark.parametrize("snapshot", [0, 1])
def test_config1_full_vector_parity(E, snapshot):
    """K=4, P=100,000, lr 0.1, mu 0.9, wd 5e-4, k=4, 10 rounds; x0 and gradients from the
    seeded recipe.  1e-6 after round one, 1e-5 after the run; mirror mode bit for bit."""
    K, P, k, rounds = 4, 100_000, 4, 10
    lr, mu, wd = 0.1, 0.9, 5e-4
    x0 = I.initial_point(P)
    worst = {}

    def check(r, eng, ref, mir):
        if r in (0, rounds - 1):
            rtol = 1e-6 if r == 0 else 1e-5
            x, v = cpu(eng.get_params()), cpu(eng.get_momentum())
            worst[r] = (assert_close_scaled(x, ref.x, rtol, f"x after round {r + 1}"),
                        assert_close_scaled(v, ref.v, rtol, f"v after round {r + 1}"))
            assert_bit_equal(x, mir.x, f"x vs mirror after round {r + 1}")
            assert_bit_equal(v, mir.v, f"v vs mirror after round {r + 1}")

    eng, ref, mir = run_both(E, K, P, lr, mu, wd, k, rounds, x0, lambda t: I.gradients(K, P, t),
                             snapshot=snapshot, check_round=check)
    assert_bit_equal(cpu(eng.get_mean()), mir.mean, "last average model")
    print("config1 worst scaled errors (x, v) by round:", worst)
    # context figures after the full run: plain relative error (unscaled, so elements near zero dominate) and the
    # distance to the fp32 mirror in units in the last place
    x = cpu(eng.get_params()).astype(np.float64)
    rel = np.abs(x - ref.x) / np.maximum(np.abs(ref.x.astype(np.float64)), 1e-300)
    ulps = np.abs(cpu(eng.get_params()).view(np.int32).astype(np.int64) - mir.x.view(np.int32).astype(np.int64))
    # the unfloored figure: plain per-element relative error over all elements that are not vanishingly small
    # (|ref| > 1e-3 * rms; the scaled bar above puts a floor of rms under |ref|, because an element that happens to lie
    # near zero after cancellation carries the absolute rounding error of its much larger summands)
    rms = np.sqrt(np.mean(ref.x.astype(np.float64) ** 2))
    big = np.abs(ref.x) > 1e-3 * rms
    print(f"config1 after the run: max relative error {rel.max():.3e}, 99.99th percentile {np.quantile(rel, 0.9999):.3e}, "
          f"max over the {big.mean():.4%} of elements with |ref| > 1e-3 rms {rel[big].max():.3e}, "
          f"max distance to the mirror {int(ulps.max())} ulp")
    assert ulps.max() == 0 and np.quantile(rel, 0.9999) < 1e-3 and rel[big].max() < 1e-2


# ----------------------------------------------------------------------------- shapes: tiles, ragged tails, misaligned rows
@pytest.mark.parametrize("K,P", [(1, 1), (1, 4099), (2, 8), (3, 7), (5, 1001), (2, 3), (16, 4096 + 4),
                                 (64, 1028), (7, 262_144 + 12), (33, 515), (128, 260),
                                 (2, 4096 + 8), (3, 1024), (4, 100_000), (1, 2048), (9, 8 * 1000),
                                 (1024, 40), (1024, 3)])          # the largest worker count the engine accepts
@pytest.mark.parametrize("snapshot", [0, 1])
def test_shapes_spanning_tiles_and_ragged_tails(E, K, P, snapshot):
    rng = np.random.default_rng(K * 1000 + P)
    k, rounds = 2, 3
    lr, mu, wd = 0.1, 0.9, 5e-4
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = (rng.standard_normal((k * rounds, K, P)) * 0.01).astype(np.float32)
    eng, ref, mir = run_both(E, K, P, lr, mu, wd, k, rounds, x0, lambda t: G[t], snapshot=snapshot)
    x, v = cpu(eng.get_params()), cpu(eng.get_momentum())
    assert_bit_equal(x, mir.x, "x vs mirror")
    assert_bit_equal(v, mir.v, "v vs mirror")
    assert_close_scaled(x, ref.x, 1e-5, "x vs ref")
    assert_close_scaled(v, ref.v, 1e-5, "v vs ref")


@pytest.mark.parametrize("seed", range(40))
def test_random_configurations_match_the_mirror_bit_for_bit(E, seed):
    """Randomised sweep over worker counts, sizes (aligned, ragged, tiny), periods, hyper-parameters,
    batch-size weights, snapshot modes, side-stream choices and the bf16 shadow: the fp32 mirror must
    be reproduced bit for bit and the reference within 1e-5."""
    rng = np.random.default_rng(1000 + seed)
    K = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 16, 17, 31, 40]))
    P = int(rng.choice([1, 2, 5, 8, 12, 64, 100, 1000, 1024, 4096, 4100, 10_007, 65_536, 100_003]))
    k, rounds = int(rng.integers(1, 5)), int(rng.integers(1, 4))
    lr = float(rng.choice([0.01, 0.05, 0.1, 0.5]))
    mu = float(rng.choice([0.0, 0.5, 0.9, 0.99]))
    wd = float(rng.choice([0.0, 1e-4, 5e-4, 1e-2]))
    M = rng.integers(1, 65, K).astype(float) if rng.random() < 0.5 else None
    snapshot = int(rng.integers(0, 2))
    side = str(rng.choice(["own", "same", "high"]))
    shadow = bool(rng.random() < 0.3)
    fuse_end = bool(rng.random() < 0.5)                 # the round's last step through cocod_local_step_end
    sweep = bool(rng.random() < 0.3)                    # kernels walking in alternating directions
    x0 = (rng.standard_normal(P) * 0.05).astype(np.float32)
    G = (rng.standard_normal((k * rounds, K, P)) * 0.02).astype(np.float32)

    eng = E.Engine(K, P, lr, mu, wd)
    eng.set_option(E.OPT_SNAPSHOT, snapshot)
    if shadow:
        eng.set_option(E.OPT_BF16_SHADOW, 1)
    if M is not None:
        eng.set_batch_sizes(M)
    if sweep:
        eng.set_option(E.OPT_SWEEP, 1)
    eng.set_params(x0)
    ref = OracleEngine(K, P, lr, mu, wd, mode="ref", batch_sizes=M)
    mir = OracleEngine(K, P, lr, mu, wd, mode="mirror", batch_sizes=M)
    ref.set_params(x0)
    mir.set_params(x0)
    side_stream = {"own": torch.cuda.Stream(), "same": torch.cuda.current_stream(),
                   "high": torch.cuda.Stream(priority=-1)}[side]
    keep = []
    for r in range(rounds):
        for o in (ref, mir):
            o.comm_begin()
        eng.comm_begin(side_stream)
        for s in range(k):
            g = G[r * k + s]
            keep.append(torch.from_numpy(g).cuda())
            if fuse_end and s == k - 1:
                eng.local_step_end(keep[-1])
            else:
                eng.local_step(keep[-1])
            ref.local_step(g)
            mir.local_step(g)
        if not fuse_end:
            eng.comm_end()
        for o in (ref, mir):
            o.comm_end()
    what = (f"K={K} P={P} k={k} rounds={rounds} lr={lr} mu={mu} wd={wd} weighted={M is not None} snapshot={snapshot} side={side} "
            f"shadow={shadow} fuse_end={fuse_end} sweep={sweep}")
    x, v = cpu(eng.get_params()), cpu(eng.get_momentum())
    assert_bit_equal(x, mir.x, "x vs mirror: " + what)
    assert_bit_equal(v, mir.v, "v vs mirror: " + what)
    assert_bit_equal(cpu(eng.get_mean()), mir.mean, "mean vs mirror: " + what)
    assert_close_scaled(x, ref.x, 1e-5, "x vs ref: " + what)
    assert_close_scaled(v, ref.v, 1e-5, "v vs ref: " + what)
    if shadow:
        assert_bit_equal(cpu(eng.bf16_shadow().float()), I.round_to_bf16(x), "shadow: " + what)


@pytest.mark.parametrize("side", ["own", "same", "high"])
@pytest.mark.parametrize("weighted", [False, True])
def test_side_stream_choices_and_weighted_mean(E, side, weighted):
    rng = np.random.default_rng(11)
    K, P, k, rounds = 6, 50_000, 3, 4
    M = rng.integers(1, 9, K).astype(float) if weighted else None
    x0 = I.initial_point(P)
    eng, ref, mir = run_both(E, K, P, 0.05, 0.9, 5e-4, k, rounds, x0, lambda t: I.gradients(K, P, t),
                             M=M, side=side)
    x = cpu(eng.get_params())
    assert_bit_equal(x, mir.x, "x vs mirror")
    assert_close_scaled(x, ref.x, 1e-5, "x vs ref")
    assert_close_scaled(cpu(eng.get_mean()), ref.mean, 1e-6, "mean vs ref")
    # line 6 preserves the weighted mean over workers
    w = np.full(K, 1 / K) if M is None else M / M.sum()
    np.testing.assert_allclose(w @ x.astype(float), w @ ref.x.astype(float), rtol=0, atol=2e-7)


def test_misaligned_gradient_pointer_takes_the_scalar_path(E):
    rng = np.random.default_rng(12)
    K, P = 3, 10_001
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    g = (rng.standard_normal(K * P + 1) * 0.01).astype(np.float32)
    gd = torch.from_numpy(g).cuda()
    view = gd[1:].view(K, P)                      # 4-byte aligned only
    assert view.data_ptr() % 16 != 0
    eng = E.Engine(K, P, 0.1, 0.9, 5e-4)
    eng.set_params(x0)
    eng.local_step(view)
    mir = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode="mirror")
    mir.set_params(x0)
    mir.local_step(g[1:].reshape(K, P))
    assert_bit_equal(cpu(eng.get_params()), mir.x)
    assert_bit_equal(cpu(eng.get_momentum()), mir.v)


# ----------------------------------------------------------------------------- degenerate cases of the method
@pytest.mark.parametrize("snapshot", [0, 1])
def test_merge_without_local_steps_is_plain_model_averaging(E, snapshot):
    rng = np.random.default_rng(13)
    K, P = 5, 3000
    X = (rng.standard_normal((K, P)) * 0.1).astype(np.float32)
    eng = E.Engine(K, P, 0.1, 0.9, 0.0)
    eng.set_option(E.OPT_SNAPSHOT, snapshot)
    eng.set_params_all(torch.from_numpy(X).cuda())
    eng.comm_begin(torch.cuda.Stream())
    eng.comm_end()
    x, m = cpu(eng.get_params()), cpu(eng.get_mean())
    for i in range(K):
        assert_bit_equal(x[i], m, f"row {i}")
    np.testing.assert_allclose(m, X.astype(float).mean(0), rtol=0, atol=3e-8)


def test_single_worker_merge_is_identity_to_rounding(E):
    rng = np.random.default_rng(14)
    P = 5000
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    G = (rng.standard_normal((6, 1, P)) * 0.01).astype(np.float32)
    eng, ref, mir = run_both(E, 1, P, 0.1, 0.9, 5e-4, 3, 2, x0, lambda t: G[t])
    # equals plain single-worker momentum SGD
    x, v = x0.astype(float), np.zeros(P)
    for t in range(6):
        v = np.float32(0.9) * v + G[t, 0] + np.float32(5e-4) * x
        x = x - np.float32(0.1) * v
    assert_close_scaled(cpu(eng.get_params())[0], x, 1e-5)
    assert_bit_equal(cpu(eng.get_params()), mir.x)


def test_pure_local_sgd_without_any_communication(E):
    rng = np.random.default_rng(15)
    K, P = 2, 777
    x0 = (rng.standard_normal(P) * 0.01).astype(np.float32)
    eng = E.Engine(K, P, 0.1, 0.0, 0.0)             # mu = wd = 0: Algorithm 1's update literally
    eng.set_params(x0)
    g = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
    eng.local_step(torch.from_numpy(g).cuda())
    want = np.float32(x0[None, :]) - np.float32(0.1) * g.astype(np.float64)
    assert_close_scaled(cpu(eng.get_params()), want, 1e-6)


# ----------------------------------------------------------------------------- boundary behaviour
def test_state_machine_and_argument_errors(E):
    eng = E.Engine(2, 16, 0.1, 0.9, 0.0)
    with pytest.raises(E.CocodError) as e:
        eng.comm_end()
    assert e.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError):
        eng.get_mean()                              # no average model exists yet
    s = torch.cuda.Stream()
    eng.comm_begin(s)
    with pytest.raises(E.CocodError) as e:
        eng.comm_begin(s)
    assert e.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError) as e:
        eng.set_params(np.zeros(16, np.float32))
    assert e.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError):
        eng.set_option(E.OPT_SNAPSHOT, 0)
    assert eng.comm_wait(2000) == E.OK
    eng.comm_end()
    with pytest.raises(E.CocodError) as e:
        eng.comm_wait(1)
    assert e.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError) as e:
        eng.set_batch_sizes([1.0, -1.0])
    assert e.value.code == E.ERR_INVALID
    with pytest.raises(E.CocodError):
        eng.set_option(99, 0)
    with pytest.raises(ValueError):
        eng.local_step(torch.zeros(2, 15, device="cuda"))
    with pytest.raises(ValueError):
        eng.local_step(torch.zeros(2, 16))          # host tensor on the device entry point
    eng.sync()
    eng.destroy()
    eng.destroy()                                   # idempotent


def test_comm_wait_reports_timeout_then_completion(E):
    """Host-side failure detection: polling the averaging with no time allowance returns TIMEOUT (or
    OK if it already finished) and never blocks; a later wait with allowance returns OK."""
    K, P = 16, 4_000_000
    eng = E.Engine(K, P, 0.1, 0.9, 0.0)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        torch.cuda._sleep(200_000_000)              # keeps the side stream busy for ~0.1 s
    eng.comm_begin(side)
    assert eng.comm_wait(0) == E.ERR_TIMEOUT
    assert eng.comm_wait(5000) == E.OK
    eng.comm_end()
    eng.sync()


def test_host_gradient_entry_point_matches_device_entry_point(E):
    K, P = 4, 300_000
    x0 = I.initial_point(P)
    a, b = E.Engine(K, P, 0.1, 0.9, 5e-4), E.Engine(K, P, 0.1, 0.9, 5e-4)
    side = torch.cuda.Stream()
    for eng in (a, b):
        eng.set_params(x0)
    for r in range(2):
        a.comm_begin(side)
        b.comm_begin(side)
        for s in range(2):
            g = I.gradients(K, P, r * 2 + s)
            a.local_step(torch.from_numpy(g).cuda())
            b.local_step_host(torch.from_numpy(g).pin_memory())
            b.sync()
        a.comm_end()
        b.comm_end()
    assert_bit_equal(cpu(a.get_params()), cpu(b.get_params()))
    assert_bit_equal(cpu(a.get_momentum()), cpu(b.get_momentum()))
    host_out = np.empty((K, P), np.float32)
    b.get_params(host_out)
    assert_bit_equal(host_out, cpu(a.get_params()))


def test_save_restore_resumes_bit_exactly(E):
    K, P, k = 3, 20_000, 2
    x0 = I.initial_point(P)
    side = torch.cuda.Stream()

    def rounds(eng, r0, r1):
        for r in range(r0, r1):
            eng.comm_begin(side)
            for s in range(k):
                eng.local_step(torch.from_numpy(I.gradients(K, P, r * k + s)).cuda())
            eng.comm_end()

    a = E.Engine(K, P, 0.1, 0.9, 5e-4)
    a.set_params(x0)
    rounds(a, 0, 6)
    b = E.Engine(K, P, 0.1, 0.9, 5e-4)
    b.set_params(x0)
    rounds(b, 0, 3)
    x, v = b.get_params().clone(), b.get_momentum().clone()
    c = E.Engine(K, P, 0.1, 0.9, 5e-4)
    c.set_params_all(x)
    c.set_momentum(v)
    rounds(c, 3, 6)
    assert_bit_equal(cpu(c.get_params()), cpu(a.get_params()))
    assert_bit_equal(cpu(c.get_momentum()), cpu(a.get_momentum()))


def test_rounds_replayed_from_a_cuda_graph_match_eager_rounds(E):
    """No call of a round blocks the host, so two rounds (one full cycle of the buffer flip) can be
    captured into a CUDA graph, side-stream averaging included, and replayed; the replays must equal
    eagerly issued rounds bit for bit."""
    K, P, k = 4, 100_000, 4
    x0 = I.initial_point(P)
    cap = torch.cuda.Stream()
    side = torch.cuda.Stream(priority=-1)
    static_g = [torch.empty((K, P), dtype=torch.float32, device="cuda") for _ in range(2 * k)]
    eager, graphed = E.Engine(K, P, 0.1, 0.9, 5e-4), E.Engine(K, P, 0.1, 0.9, 5e-4)
    for eng in (eager, graphed):
        eng.set_params(x0)
    graphed.sync()
    graphed.set_stream(cap)

    def two_rounds(eng):
        for r in range(2):
            eng.comm_begin(side)
            for s in range(k):
                eng.local_step(static_g[r * k + s])
            eng.comm_end()

    def load(block):
        for i, g in enumerate(static_g):
            g.copy_(torch.from_numpy(I.gradients(K, P, block * 2 * k + i)))

    load(0)
    torch.cuda.synchronize()
    with torch.cuda.stream(cap):
        two_rounds(graphed)                          # warm-up on the capture stream
    two_rounds(eager)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    load(1)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=cap):
        two_rounds(graphed)
    for block in (1, 2, 3):
        load(block)
        torch.cuda.synchronize()
        graph.replay()
        two_rounds(eager)
        torch.cuda.synchronize()
        assert_bit_equal(cpu(graphed.get_params()), cpu(eager.get_params()), f"x after block {block}")
        assert_bit_equal(cpu(graphed.get_momentum()), cpu(eager.get_momentum()), f"v after block {block}")


@pytest.mark.parametrize("K,P,snapshot", [(3, 1001, 1), (4, 4100, 0), (2, 8 * 1000, 1), (16, 65_536 + 64, 1)])
def test_bf16_shadow_tracks_the_master_copy_on_every_path(E, K, P, snapshot):
    """With the bf16 shadow on, every kernel that writes x (local step, merge; vector and scalar
    paths, both snapshot modes) also writes bf16(x): after each call the shadow equals the master
    copy rounded to nearest even, and the fp32 results are unchanged by the option."""
    rng = np.random.default_rng(P)
    x0 = (rng.standard_normal(P) * 0.05).astype(np.float32)
    eng = E.Engine(K, P, 0.1, 0.9, 5e-4)
    eng.set_option(E.OPT_SNAPSHOT, snapshot)
    eng.set_option(E.OPT_BF16_SHADOW, 1)
    eng.set_params(x0)
    mir = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode="mirror")
    mir.set_params(x0)
    side = torch.cuda.Stream()

    def check(tag):
        x = cpu(eng.get_params())
        assert_bit_equal(x, mir.x, f"x {tag}")
        assert_bit_equal(cpu(eng.bf16_shadow().float()), I.round_to_bf16(x), f"shadow {tag}")

    check("after set_params")
    for r in range(2):
        eng.comm_begin(side)
        mir.comm_begin()
        for s in range(2):
            g = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
            eng.local_step(torch.from_numpy(g).cuda())
            mir.local_step(g)
            check(f"after step {r}.{s}")
        eng.comm_end()
        mir.comm_end()
        check(f"after merge {r}")
    X = (rng.standard_normal((K, P)) * 0.05).astype(np.float32)
    eng.set_params_all(X)
    mir.set_params_all(X)
    check("after set_params_all")
    eng.set_option(E.OPT_BF16_SHADOW, 0)
    with pytest.raises(E.CocodError):
        eng.bf16_shadow()


def test_switching_the_compute_stream_keeps_work_ordered(E):
    K, P = 4, 200_000
    x0 = I.initial_point(P)
    a, b = torch.cuda.Stream(), torch.cuda.Stream()
    eng = E.Engine(K, P, 0.1, 0.9, 5e-4)
    mir = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode="mirror")
    eng.set_params(x0)
    mir.set_params(x0)
    side = torch.cuda.Stream()
    gs = [torch.from_numpy(I.gradients(K, P, t)).cuda() for t in range(6)]
    torch.cuda.synchronize()
    for r, stream in enumerate([a, b, a]):
        eng.set_stream(stream)                       # later work must wait for what the old stream still runs
        eng.comm_begin(side)
        mir.comm_begin()
        for s in range(2):
            eng.local_step(gs[2 * r + s])
            mir.local_step(cpu(gs[2 * r + s]))
        eng.comm_end()
        mir.comm_end()
    eng.sync()
    assert_bit_equal(cpu(eng.get_params()), mir.x)


@pytest.mark.parametrize("K,P,weighted", [(4, 100_000, False), (5, 1001, True), (16, 65_536 + 8, True), (2, 7, False)])
def test_sequential_schemes_local_sgd_and_ssgd(E, K, P, weighted):
    """The two schemes the paper compares against, on the same kernels: Local-SGD (k local steps, then
    blocking model averaging) and S-SGD (gradient averaging every step), against the oracle."""
    rng = np.random.default_rng(K + P)
    M = rng.integers(1, 9, K).astype(float) if weighted else None
    x0 = (rng.standard_normal(P) * 0.05).astype(np.float32)
    G = (rng.standard_normal((6, K, P)) * 0.02).astype(np.float32)
    for scheme in ("local_sgd", "ssgd"):
        eng = E.Engine(K, P, 0.1, 0.9, 5e-4)
        ref = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode="ref", batch_sizes=M)
        mir = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode="mirror", batch_sizes=M)
        if M is not None:
            eng.set_batch_sizes(M)
        eng.set_params(x0)
        ref.set_params(x0)
        mir.set_params(x0)
        for t in range(6):
            gd = torch.from_numpy(G[t]).cuda()
            if scheme == "ssgd":
                eng.ssgd_step(gd)
                ref.ssgd_step(G[t])
                mir.ssgd_step(G[t])
            else:
                eng.local_step(gd)
                ref.local_step(G[t])
                mir.local_step(G[t])
                if t % 2 == 1:                     # period k = 2
                    eng.local_sgd_average()
                    ref.local_sgd_average()
                    mir.local_sgd_average()
        x, v = cpu(eng.get_params()), cpu(eng.get_momentum())
        assert_bit_equal(x, mir.x, f"{scheme}: x vs mirror")
        assert_bit_equal(v, mir.v, f"{scheme}: v vs mirror")
        assert_close_scaled(x, ref.x, 1e-5, f"{scheme}: x vs ref")
        if scheme == "ssgd":
            for i in range(1, K):
                assert_bit_equal(x[i], x[0], "replicas stay identical under S-SGD")
        assert eng.step_count == 6
    eng.comm_begin(torch.cuda.Stream())
    with pytest.raises(E.CocodError):
        eng.ssgd_step(gd)
    with pytest.raises(E.CocodError):
        eng.local_sgd_average()
    eng.comm_end()


def test_learning_rate_schedule_and_profile_records(E):
    K, P = 2, 4096
    eng = E.Engine(K, P, 0.1, 0.9, 0.0)
    mir = OracleEngine(K, P, 0.1, 0.9, 0.0, mode="mirror")
    x0 = I.initial_point(P)
    eng.set_params(x0)
    mir.set_params(x0)
    eng.set_option(E.OPT_PROFILE, 1)
    side = torch.cuda.Stream()
    for r, lr in enumerate([0.1, 0.01]):
        eng.set_lr(lr)
        mir.set_lr(lr)
        eng.comm_begin(side)
        mir.comm_begin()
        g = I.gradients(K, P, r)
        eng.local_step(torch.from_numpy(g).cuda())
        mir.local_step(g)
        eng.comm_end()
        mir.comm_end()
    assert_bit_equal(cpu(eng.get_params()), mir.x)
    recs = eng.profile_records()
    kinds = [E.KERNEL_NAMES[k] for k, _, _ in recs]
    assert kinds.count("local_step") == 2 and kinds.count("mean") == 2 and kinds.count("merge") == 2
    assert all(b >= a for _, a, b in recs)
    assert eng.launch_count >= 7


# ----------------------------------------------------------------------------- the four kernels on caller buffers
def test_stateless_kernels_against_oracle_pieces(E):
    rng = np.random.default_rng(16)
    K, P = 9, 12_345 * 4
    X = (rng.standard_normal((K, P)) * 0.1).astype(np.float32)
    S = (rng.standard_normal((K, P)) * 0.1).astype(np.float32)
    V = (rng.standard_normal((K, P)) * 0.02).astype(np.float32)
    G = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
    mir = OracleEngine(K, P, 0.1, 0.9, 5e-4, mode="mirror")
    mir.x[:], mir.v[:] = X, V
    mir.local_step(G)
    x, v, g = (torch.from_numpy(a).cuda() for a in (X, V, G))
    x_out = torch.empty_like(x)
    E.kernel_local_step(x, x_out, v, g, 0.1, 0.9, 5e-4)
    assert_bit_equal(cpu(x_out), mir.x)
    assert_bit_equal(cpu(v), mir.v)
    assert_bit_equal(cpu(x), X, "out-of-place step must not touch x_in")
    snap = torch.empty_like(x)
    E.kernel_snapshot(x, snap)
    assert_bit_equal(cpu(snap), X)
    # mean / merge
    mir2 = OracleEngine(K, P, 0.1, 0.9, 0.0, mode="mirror")
    mir2.x[:] = S
    mir2.comm_begin()
    mir2.x[:] = X
    mir2.comm_end()
    sd, mean = torch.from_numpy(S).cuda(), torch.empty(P, dtype=torch.float32, device="cuda")
    E.kernel_mean(sd, mean)
    assert_bit_equal(cpu(mean), mir2.mean)
    xd = torch.from_numpy(X).cuda()
    E.kernel_merge(xd, sd, mean)
    assert_bit_equal(cpu(xd), mir2.x)


def test_buffers_next_to_engine_inputs_are_untouched(E):
    """Guard bands around a caller-owned gradient buffer stay intact (no out-of-range access)."""
    K, P = 3, 4097
    pad = 1024
    big = torch.full((K * P + 2 * pad,), float("nan"), device="cuda")
    g = big[pad:pad + K * P].view(K, P)
    g.copy_(torch.from_numpy(I.gradients(K, P, 0)).cuda())
    eng = E.Engine(K, P, 0.1, 0.9, 5e-4)
    eng.set_params(I.initial_point(P))
    eng.comm_begin(torch.cuda.Stream())
    eng.local_step(g)
    eng.comm_end()
    eng.sync()
    assert torch.isnan(big[:pad]).all() and torch.isnan(big[pad + K * P:]).all()
    assert torch.isfinite(eng.get_params()).all()


def test_a_request_beyond_the_device_memory_fails_cleanly(E):
    """cocod_create with buffers that cannot exist (256 GB each): out-of-memory error code, nothing leaked,
    and the device is as usable as before."""
    free_before = torch.cuda.mem_get_info()[0]
    with pytest.raises(E.CocodError) as e:
        E.Engine(16, 4_000_000_000, 0.1, 0.9, 0.0)
    assert e.value.code == E.ERR_OOM
    assert abs(torch.cuda.mem_get_info()[0] - free_before) < (64 << 20)
    eng = E.Engine(2, 1024, 0.1, 0.0, 0.0)
    eng.set_params(np.ones(1024, np.float32))
    eng.local_step(torch.ones(2, 1024, device="cuda"))
    assert np.allclose(cpu(eng.get_params()), 0.9)
    eng.destroy()


# ----------------------------------------------------------------------------- measurement options change no value
@pytest.mark.parametrize("K,P,shadow", [(16, 200_000, False), (5, 100_008, True), (3, 1001, False)])
def test_alternating_sweep_and_device_time_stamps_change_no_value(E, K, P, shadow):
    """COCOD_OPT_SWEEP lets consecutive kernels walk the vector in alternating directions, COCOD_OPT_PROFILE lets
    them stamp their start and end on the GPU's clock: the models, momenta, averages (and bf16 copies) must equal
    the plain run bit for bit, and the stamps must be ordered and cover every recorded kernel that takes them."""
    k, rounds = 3, 3
    x0 = I.initial_point(P)
    side = torch.cuda.Stream(priority=-1)
    engines = [E.Engine(K, P, 0.1, 0.9, 5e-4) for _ in range(2)]
    for eng in engines:
        if shadow:
            eng.set_option(E.OPT_BF16_SHADOW, 1)
        eng.set_params(x0)
    engines[1].set_option(E.OPT_SWEEP, 1)
    engines[1].set_option(E.OPT_PROFILE, 1)
    engines[1].profile_reset()
    for r in range(rounds):
        for eng in engines:
            eng.comm_begin(side)
        for s in range(k):
            g = torch.from_numpy(I.gradients(K, P, r * k + s)).cuda()
            for eng in engines:
                eng.local_step(g)
        for eng in engines:
            eng.comm_end()
    a, b = engines
    assert_bit_equal(cpu(b.get_params()), cpu(a.get_params()), "x")
    assert_bit_equal(cpu(b.get_momentum()), cpu(a.get_momentum()), "v")
    assert_bit_equal(cpu(b.get_mean()), cpu(a.get_mean()), "average")
    if shadow:
        assert torch.equal(a.bf16_shadow().view(torch.int16), b.bf16_shadow().view(torch.int16))
    events = b.profile_records()
    stamps = b.profile_device_records()
    assert len(events) == rounds * (k + 2)
    if P % 4 == 0:                                   # the vectorised kernels take stamps, the scalar fall-backs do not
        assert len(stamps) == len(events)
        for kind, t0, t1 in stamps:
            assert 0.0 <= t0 < t1 < 1e4
        # stream order on the compute stream: every local step / merge starts after its predecessor started
        comp = [(t0, t1) for kind, t0, t1 in stamps if E.KERNEL_NAMES[kind] != "mean"]
        assert all(comp[i][0] <= comp[i + 1][0] for i in range(len(comp) - 1))
    else:                                            # the flat local step still has a vectorised body; mean and merge do not
        assert len(stamps) == rounds * k and all(E.KERNEL_NAMES[kind] == "local_step" for kind, _, _ in stamps)


# ----------------------------------------------------------------------------- fusion variant: last step + merge
@pytest.mark.parametrize("K,P,k", [(16, 200_000, 2), (4, 100_000, 4), (5, 100_008, 1), (3, 1001, 2), (1, 4096, 3),
                                   (64, 1032, 2), (2, 8, 1), (9, 8 * 1000, 3), (7, 262_144 + 12, 2)])
@pytest.mark.parametrize("snapshot", [0, 1])
def test_last_step_fused_with_the_merge_equals_the_two_calls_and_the_oracle(E, K, P, k, snapshot):
    """cocod_local_step_end = the round's last iteration of Step II and line 6 in one pass.  Against the oracle (ref
    at 1e-6 after one round / 1e-5 after the run, fp32 mirror bit for bit) and against an engine that makes the two
    calls (bit for bit: x, v, average, bf16 copy), over rounds of k steps (k = 1: the stepped x aliases the stored copy
    under the flip), unequal batch sizes, shapes that take the fused kernel and shapes that fall back to the two kernels."""
    rounds, lr, mu, wd = 3, 0.1, 0.9, 5e-4
    x0 = I.initial_point(P)
    M = np.arange(1, K + 1, dtype=np.float64) if K in (5, 9) else None
    fusedE, plainE = E.Engine(K, P, lr, mu, wd), E.Engine(K, P, lr, mu, wd)
    ref = OracleEngine(K, P, lr, mu, wd, mode="ref", batch_sizes=M)
    mir = OracleEngine(K, P, lr, mu, wd, mode="mirror", batch_sizes=M)
    for eng in (fusedE, plainE):
        eng.set_option(E.OPT_SNAPSHOT, snapshot)
        eng.set_option(E.OPT_BF16_SHADOW, 1)
        if M is not None:
            eng.set_batch_sizes(M)
        eng.set_params(torch.from_numpy(x0).cuda())
    ref.set_params(x0)
    mir.set_params(x0)
    side = torch.cuda.Stream(priority=-1)
    with pytest.raises(E.CocodError) as err:
        fusedE.local_step_end(torch.zeros((K, P), dtype=torch.float32, device="cuda"))      # no round in flight
    assert err.value.code == E.ERR_STATE
    for r in range(rounds):
        for eng in (fusedE, plainE):
            eng.comm_begin(side)
        ref.comm_begin()
        mir.comm_begin()
        for s in range(k):
            g = I.gradients(K, P, r * k + s)
            gd = torch.from_numpy(g).cuda()
            if s < k - 1:
                fusedE.local_step(gd)
            else:
                fusedE.local_step_end(gd)
            plainE.local_step(gd)
            ref.local_step(g)
            mir.local_step(g)
        plainE.comm_end()
        ref.comm_end()
        mir.comm_end()
        what = f"round {r + 1}"
        for got, want, name in ((fusedE.get_params(), plainE.get_params(), "x"), (fusedE.get_momentum(), plainE.get_momentum(), "v"),
                                (fusedE.get_mean(), plainE.get_mean(), "average")):
            assert torch.equal(got.view(torch.int32), want.view(torch.int32)), f"{name}, {what}"
        assert torch.equal(fusedE.bf16_shadow().view(torch.int16), plainE.bf16_shadow().view(torch.int16)), f"bf16 copy, {what}"
        assert_bit_equal(cpu(fusedE.get_params()), mir.x, f"x vs mirror, {what}")
        assert_bit_equal(cpu(fusedE.get_momentum()), mir.v, f"v vs mirror, {what}")
        rtol = 1e-6 if r == 0 else 1e-5
        assert_close_scaled(cpu(fusedE.get_params()), ref.x, rtol, f"x vs ref, {what}")
        assert_close_scaled(cpu(fusedE.get_momentum()), ref.v, rtol, f"v vs ref, {what}")
    assert fusedE.step_count == plainE.step_count == rounds * k
    np.testing.assert_array_equal(cpu(fusedE.bf16_shadow().float()), I.round_to_bf16(cpu(fusedE.get_params())))


def test_rounds_ending_in_the_fused_call_replay_from_a_cuda_graph(E):
    """Two rounds whose last step goes through cocod_local_step_end (which waits, on the stream, for the side stream's
    mean) captured into a CUDA graph and replayed: equal to eagerly issued explicit rounds, bit for bit."""
    K, P, k = 4, 100_000, 3
    x0 = I.initial_point(P)
    cap, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    static_g = [torch.from_numpy(I.gradients(K, P, t)).cuda() for t in range(2 * k)]
    eager, graphed = E.Engine(K, P, 0.1, 0.9, 5e-4), E.Engine(K, P, 0.1, 0.9, 5e-4)
    for eng in (eager, graphed):
        eng.set_params(x0)
    graphed.sync()
    graphed.set_stream(cap)

    def two_rounds(eng, fused_end):
        for r in range(2):
            eng.comm_begin(side)
            for s in range(k):
                if fused_end and s == k - 1:
                    eng.local_step_end(static_g[r * k + s])
                else:
                    eng.local_step(static_g[r * k + s])
            if not fused_end:
                eng.comm_end()

    with torch.cuda.stream(cap):
        two_rounds(graphed, True)                    # warm-up on the capture stream
    two_rounds(eager, False)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=cap):
        two_rounds(graphed, True)
    for _ in range(3):
        graph.replay()
        two_rounds(eager, False)
        torch.cuda.synchronize()
        assert_bit_equal(cpu(graphed.get_params()), cpu(eager.get_params()), "x")
        assert_bit_equal(cpu(graphed.get_momentum()), cpu(eager.get_momentum()), "v")
    graphed.sync()
    graphed.set_stream(torch.cuda.current_stream())
