"""Workers spread over several engines ("GPUs"): the two ways of completing Step I's mean across
them, on ONE device.

No kernel here waits on another.  The ranks are either several engines inside this process whose
work is queued on one device in program order (the exchange between them is emulated by plain
stream-ordered work), or two processes on the same device that order themselves with host barriers.

Bars: the gather form sums in worker order, so it must equal the oracle's fp32 mirror of the
single-engine run bit for bit however the workers are spread; the all-reduce form changes the order
of the sum over ranks and is held to the fp32 tolerances (1e-6 scaled after one round, 1e-5 after the
run) against the oracle's reference mode.
"""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import cocod_oracle as O
from oracle.cocod_oracle import OracleEngine
from paper_1906_12043_b200 import inputs as I
from paper_1906_12043_b200.sharded import shard_workers

pytestmark = pytest.mark.gpu
LR, MU, WD = 0.1, 0.9, 5e-4


@pytest.fixture(scope="module")
def E():
    from paper_1906_12043_b200 import build, engine
    build.build()
    engine.load()
    return engine


def cpu(t):
    return t.detach().cpu().numpy()


def assert_bit_equal(got, ref, what=""):
    got = np.ascontiguousarray(got, np.float32).view(np.uint32)
    ref = np.ascontiguousarray(ref, np.float32).view(np.uint32)
    bad = np.nonzero(got != ref)
    assert bad[0].size == 0, f"{what}: {bad[0].size} elements differ, first at {[b[0] for b in bad]}"


def assert_close_scaled(got, ref, rtol, what=""):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    scale = np.maximum(np.abs(ref), np.sqrt(np.mean(ref ** 2)))
    worst = float((np.abs(got - ref) / np.maximum(scale, 1e-300)).max())
    assert worst <= rtol, f"{what}: max scaled error {worst:.3e} > {rtol:.1e}"


def oracle_run(K, P, k, rounds, M, mode, after_round=None):
    o = OracleEngine(K, P, LR, MU, WD, mode=mode, batch_sizes=M)
    o.set_params(I.initial_point(P))
    o.run(lambda t: I.gradients(K, P, t), k, rounds, on_round=after_round)
    return o


def address_table(tensors):
    return torch.tensor([t.data_ptr() for t in tensors], dtype=torch.int64, device="cuda")


# ----------------------------------------------------------------------------- the gather kernel by itself
@pytest.mark.parametrize("K,P,weighted,vec", [
    (1, 4096, False, 4), (3, 4 * 1001, True, 4), (8, 4 * 50_000, False, 4),
    (16, 4 * 50_001, False, 4), (19, 4 * 7777, True, 4), (16, 10_007, False, 1),
    (5, 999, True, 1), (1, 8 * 999, False, 8), (2, 8 * 40_001, True, 8), (3, 8 * 5_000, False, 8),
    (4, 8 * 30_000, True, 8), (16, 8 * 30_000, False, 8),
])
def test_gather_kernel_equals_the_mirror_mean_with_rows_in_separate_allocations(E, K, P, weighted, vec):
    rng = np.random.default_rng(K * 1000 + P)
    S = (rng.standard_normal((K, P)) * 0.1).astype(np.float32)
    M = rng.integers(1, 9, K).astype(np.float64) * 32 if weighted else None
    expect = np.zeros(P, np.float32)
    Mp = None if M is None else M.ctypes.data_as(O.ctypes.POINTER(O.ctypes.c_double))
    O.lib().oracle_mean_mirror(K, P, S.ctypes.data_as(O.ctypes.POINTER(O.ctypes.c_float)), Mp,
                               expect.ctypes.data_as(O.ctypes.POINTER(O.ctypes.c_float)))
    rows = [torch.from_numpy(S[i].copy()).cuda() for i in range(K)]          # K separate allocations
    G = 3
    outs = [torch.full((P,), float("nan"), device="cuda") for _ in range(G)]
    w = None if M is None else torch.from_numpy((M / M.sum()).astype(np.float32)).cuda()
    unit = vec
    lo, hi = (P // 3) // unit * unit, (2 * P // 3) // unit * unit             # a share in the middle
    E.kernel_mean_gather(address_table(rows), lo, hi, address_table(outs), w=w, vec=vec)
    torch.cuda.synchronize()
    for q in range(G):
        got = cpu(outs[q])
        assert_bit_equal(got[lo:hi], expect[lo:hi], f"out {q}")
        assert np.isnan(got[:lo]).all() and np.isnan(got[hi:]).all(), "columns outside the share were written"
    # the shares of all ranks tile the buffer
    for r in range(G):
        units = P // unit
        a, b = units * r // G * unit, (units * (r + 1) // G * unit if r < G - 1 else P)
        b = b // unit * unit
        E.kernel_mean_gather(address_table(rows), a, b, address_table(outs), w=w, vec=vec)
    torch.cuda.synchronize()
    assert_bit_equal(cpu(outs[1])[:P // unit * unit], expect[:P // unit * unit])
    with pytest.raises(E.CocodError) as e:
        E.kernel_mean_gather(address_table(rows), 2, 8, address_table(outs), vec=4)
    assert e.value.code == E.ERR_INVALID


# ----------------------------------------------------------------------------- several engines in this process
def virtual_ranks(E, K_global, G, P, M, attach):
    engs = []
    for r in range(G):
        first, count = shard_workers(K_global, G, r)
        e = E.Engine(count, P, LR, MU, WD)
        e.set_shard(K_global, first, M)
        e.set_params(torch.from_numpy(I.initial_point(P)).cuda())
        engs.append(e)
    if attach:
        blobs = [e.ipc_export() for e in engs]
        for r, e in enumerate(engs):
            e.ipc_attach(r, blobs)
    return engs


def drive(E, engs, K_global, P, k, rounds, form, after_round=None, fuse_end=False):
    """Algorithm 1 over all engines; everything is queued on one device in program order.  fuse_end: the round's last
    local step and line 6 through cocod_local_step_end instead of the two calls."""
    G = len(engs)
    sides = [torch.cuda.Stream() for _ in engs]
    bounds = [shard_workers(K_global, G, r) for r in range(G)]
    keep = []
    for r in range(rounds):
        for e, s in zip(engs, sides):
            e.comm_begin(s)
        if form == "allreduce":
            # the all-reduce, emulated: once every partial sum is complete, every engine's buffer gets the total
            torch.cuda.synchronize()
            total = torch.stack([e.mean_buffer() for e in engs]).sum(0)
            for e, s in zip(engs, sides):
                with torch.cuda.stream(s):
                    e.mean_buffer().copy_(total)
        else:
            torch.cuda.synchronize()          # barrier 1: every engine's stored copies exist
            for e in engs:
                e.comm_gather()
            torch.cuda.synchronize()          # barrier 2: every engine's columns have arrived everywhere
        for e in engs:
            e.comm_exchanged()
        for s in range(k):
            g = I.gradients(K_global, P, r * k + s)
            for e, (first, count) in zip(engs, bounds):
                gd = torch.from_numpy(np.ascontiguousarray(g[first:first + count])).cuda()
                keep.append(gd)
                if fuse_end and s == k - 1:
                    e.local_step_end(gd)
                else:
                    e.local_step(gd)
        if not fuse_end:
            for e in engs:
                e.comm_end()
        if after_round is not None:
            torch.cuda.synchronize()
            after_round(r, np.concatenate([cpu(e.get_params()) for e in engs], 0))
    torch.cuda.synchronize()
    x = np.concatenate([cpu(e.get_params()) for e in engs], 0)
    v = np.concatenate([cpu(e.get_momentum()) for e in engs], 0)
    return x, v


def close_all(engs, attached):
    for e in engs:
        e.sync()
    if attached:
        for e in engs:
            e.ipc_detach()
    for e in engs:
        e.destroy()


@pytest.mark.parametrize("K_global,G,P,weighted", [
    (16, 2, 4 * 30_011, False), (16, 8, 4 * 30_011, False), (16, 16, 4 * 5_003, False),
    (5, 2, 4 * 9_001, True), (19, 4, 10_007, True), (4, 4, 100_000, False), (3, 1, 4 * 777, False),
])
def test_gather_form_equals_the_single_engine_mirror_bit_for_bit(E, K_global, G, P, weighted):
    k, rounds = 2, 3
    M = [32.0 * (1 + (i * 7) % 5) for i in range(K_global)] if weighted else None
    mir = oracle_run(K_global, P, k, rounds, M, "mirror")
    engs = virtual_ranks(E, K_global, G, P, M, attach=True)
    x, v = drive(E, engs, K_global, P, k, rounds, "gather", fuse_end=(G in (2, 4)))      # some spreads through the fused call
    assert_bit_equal(x, mir.x, "x")
    assert_bit_equal(v, mir.v, "v")
    assert_bit_equal(cpu(engs[-1].get_mean()), mir.mean, "average model")
    close_all(engs, True)


@pytest.mark.parametrize("K_global,G,P,weighted", [
    (16, 2, 4 * 30_011, False), (16, 4, 4 * 30_011, True), (5, 2, 10_007, True), (64, 8, 4 * 4_001, False),
])
def test_allreduce_form_meets_the_fp32_tolerances_against_the_reference_oracle(E, K_global, G, P, weighted):
    k, rounds = 2, 4
    M = [32.0 * (1 + (i * 3) % 4) for i in range(K_global)] if weighted else None
    first_round = {}
    ref = oracle_run(K_global, P, k, rounds, M, "ref",
                     after_round=lambda r, o: first_round.setdefault("x", o.x.copy()) if r == 0 else None)
    engs = virtual_ranks(E, K_global, G, P, M, attach=False)
    got_first = {}
    x, v = drive(E, engs, K_global, P, k, rounds, "allreduce",
                 after_round=lambda r, xs: got_first.setdefault("x", xs) if r == 0 else None)
    assert_close_scaled(got_first["x"], first_round["x"], 1e-6, "x after one round")
    assert_close_scaled(x, ref.x, 1e-5, "x after the run")
    assert_close_scaled(v, ref.v, 1e-5, "v after the run")
    if K_global == 16 and G == 2 and not weighted:
        # two blocks of 8 workers, scaled by a power of two: the same fp32 operations as one engine
        mir = oracle_run(K_global, P, k, rounds, M, "mirror")
        assert_bit_equal(x, mir.x)
    close_all(engs, False)


def test_partial_sum_carries_the_global_weights(E):
    """What cocod_comm_begin leaves in the average buffer of a sharded engine."""
    K_global, P = 7, 4 * 501
    M = [32.0, 64.0, 96.0, 32.0, 128.0, 64.0, 32.0]
    rng = np.random.default_rng(3)
    X = (rng.standard_normal((K_global, P)) * 0.1).astype(np.float32)
    for first, count in ((0, 3), (3, 4), (2, 1)):
        for Mg in (None, M):
            e = E.Engine(count, P, LR, MU, WD)
            e.set_shard(K_global, first, Mg)
            e.set_params_all(torch.from_numpy(X[first:first + count].copy()).cuda())
            s = torch.cuda.Stream()
            e.comm_begin(s)
            s.synchronize()
            w = np.full(K_global, 1.0 / K_global) if Mg is None else np.asarray(Mg) / np.sum(Mg)
            expect = (w[first:first + count, None] * X[first:first + count].astype(np.float64)).sum(0)
            assert_close_scaled(cpu(e.mean_buffer()), expect, 1e-6, f"partial sum of workers {first}..{first + count}")
            e.comm_exchanged()
            e.comm_end()
            e.sync()
            e.destroy()


def test_sharded_state_machine_and_argument_errors(E):
    P = 64
    e = E.Engine(2, P, LR, MU, WD)
    for bad in ((1, 0), (1025, 0), (4, 3), (4, -1)):            # fewer workers than held; too many; block sticks out
        with pytest.raises(E.CocodError) as err:
            e.set_shard(*bad)
        assert err.value.code == E.ERR_INVALID
    with pytest.raises(E.CocodError) as err:
        e.set_shard(4, 0, [1.0, 2.0, 0.0, 1.0])
    assert err.value.code == E.ERR_INVALID
    with pytest.raises(E.CocodError) as err:
        e.ipc_export()                                           # not sharded yet
    assert err.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError) as err:
        e.comm_exchanged()
    assert err.value.code == E.ERR_STATE
    e.set_shard(4, 2)
    for call in (e.local_sgd_average, lambda: e.ssgd_step(torch.zeros(2, P, device="cuda")),
                 lambda: e.set_batch_sizes([1.0, 2.0]), e.comm_gather):
        with pytest.raises(E.CocodError) as err:
            call()
        assert err.value.code == E.ERR_STATE
    s = torch.cuda.Stream()
    e.comm_begin(s)
    with pytest.raises(E.CocodError) as err:
        e.comm_end()                                             # the mean over the GPUs is not complete
    assert err.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError) as err:
        e.comm_wait(1)
    assert err.value.code == E.ERR_STATE
    with pytest.raises(E.CocodError) as err:
        e.set_shard(0, 0)
    assert err.value.code == E.ERR_STATE
    e.comm_exchanged()
    with pytest.raises(E.CocodError) as err:
        e.comm_exchanged()                                       # once per round
    assert err.value.code == E.ERR_STATE
    assert e.comm_wait(2000) == E.OK
    e.comm_end()
    # address blobs that do not tile the workers, or come from a differently shaped engine, are refused
    other = E.Engine(2, P, LR, MU, WD)
    other.set_shard(4, 2)                                        # overlaps e instead of starting at 0
    with pytest.raises(E.CocodError) as err:
        e.ipc_attach(1, [other.ipc_export(), e.ipc_export()])
    assert err.value.code == E.ERR_INVALID
    other.set_shard(4, 0)
    wrong_p = E.Engine(2, P + 4, LR, MU, WD)
    wrong_p.set_shard(4, 0)
    with pytest.raises(E.CocodError) as err:
        e.ipc_attach(1, [wrong_p.ipc_export(), e.ipc_export()])
    assert err.value.code == E.ERR_INVALID
    with pytest.raises(E.CocodError) as err:
        e.ipc_attach(0, [other.ipc_export(), e.ipc_export()])    # this engine is rank 1, not 0
    assert err.value.code == E.ERR_INVALID
    e.ipc_attach(1, [other.ipc_export(), e.ipc_export()])
    with pytest.raises(E.CocodError) as err:
        e.set_shard(0, 0)                                        # not while peers are attached
    assert err.value.code == E.ERR_STATE
    e.ipc_detach()
    e.set_shard(0, 0)                                            # back to a plain engine
    e.comm_begin(s)
    e.comm_end()
    for x in (e, other, wrong_p):
        x.sync()
        x.destroy()


# ----------------------------------------------------------------------------- the distributed wrapper itself
def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("exchange", ["allreduce", "gather"])
def test_wrapper_over_a_one_process_nccl_group_equals_the_plain_engine(E, exchange):
    """world_size 1 on the one GPU: the collective calls, their stream ordering and the address
    exchange all run; the result must be the plain engine's, bit for bit."""
    import torch.distributed as dist
    from paper_1906_12043_b200.sharded import WorkerShardedEngine
    K, P, k, rounds = 6, 4 * 20_003, 3, 3
    mir = oracle_run(K, P, k, rounds, None, "mirror")
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        eng = WorkerShardedEngine(K, P, LR, MU, WD, exchange=exchange, sync="stream")
        eng.set_params(torch.from_numpy(I.initial_point(P)).cuda())
        side = torch.cuda.Stream()
        keep = []
        for r in range(rounds):
            eng.comm_begin(side)
            for s in range(k):
                keep.append(torch.from_numpy(I.gradients(K, P, r * k + s)).cuda())
                eng.local_step(keep[-1])
            eng.comm_end()
        eng.sync()
        assert_bit_equal(cpu(eng.get_params()), mir.x)
        assert_bit_equal(cpu(eng.get_momentum()), mir.v)
        eng.close()
    finally:
        dist.destroy_process_group()


def _two_process_worker(rank, world, port, K_global, P, k, rounds, M, exchange, out_dir):
    import torch.distributed as dist
    from paper_1906_12043_b200.sharded import WorkerShardedEngine
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    eng = WorkerShardedEngine(K_global, P, LR, MU, WD, batch_sizes=M, exchange=exchange, sync="host")
    eng.set_params(torch.from_numpy(I.initial_point(P)).cuda())
    side = torch.cuda.Stream()
    keep = []
    for r in range(rounds):
        eng.comm_begin(side)
        for s in range(k):
            g = I.gradients(K_global, P, r * k + s)[eng.first:eng.first + eng.K]
            keep.append(torch.from_numpy(np.ascontiguousarray(g)).cuda())
            eng.local_step(keep[-1])
        eng.comm_end()
    eng.sync()
    np.save(os.path.join(out_dir, f"x{rank}.npy"), cpu(eng.get_params()))
    eng.close()
    dist.destroy_process_group()


@pytest.mark.parametrize("K_global,M", [(16, None), (5, [32.0, 64.0, 128.0, 32.0, 256.0])])
def test_two_processes_on_one_device_exchange_addresses_and_gather(E, tmp_path, K_global, M):
    """Two processes, each with its own engine on the same device: the inter-process memory handles
    are opened for real and each process's kernel reads the other's stored copies and writes the
    other's average buffer.  Ordering between the processes is by host barriers only."""
    import torch.multiprocessing as mp
    P, k, rounds, world = 4 * 25_003, 2, 3, 2
    mp.spawn(_two_process_worker, args=(world, _free_port(), K_global, P, k, rounds, M, "gather", str(tmp_path)),
             nprocs=world, join=True)
    mir = oracle_run(K_global, P, k, rounds, M, "mirror")
    got = np.concatenate([np.load(tmp_path / f"x{r}.npy") for r in range(world)], 0)
    assert_bit_equal(got, mir.x)
