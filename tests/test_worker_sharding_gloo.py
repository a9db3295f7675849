"""Workers spread over processes (gloo, world_size 2, CPU): the host logic of
``paper_1906_12043_b200.sharded`` -- which workers live where, the global weights, the order of
what is queued per round, the exchange of address blobs -- driven with a host stand-in for the
CUDA engine.  Whatever the spread, the run must reproduce Algorithm 1 over all K workers as the
oracle computes it in one piece."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle.cocod_oracle import OracleEngine
from paper_1906_12043_b200 import inputs as I
from paper_1906_12043_b200.sharded import WorkerShardedEngine, shard_workers

P, k, ROUNDS = 203, 2, 3
LR, MU, WD = 0.1, 0.9, 5e-4


class HostEngine:
    """Test double with the sharded engine's calls: local step and merge are the oracle's, the
    partial sum is written out in fp64, and "peer memory" is an all-gather over the group."""

    def __init__(self, K, P_, lr, mu, wd):
        self.K, self.P = K, P_
        self.o = OracleEngine(K, P_, lr, mu, wd, mode="ref")
        self.phase = "idle"
        self.log = []
        self.attached = None

    def set_shard(self, K_global, first, M_global):
        self.K_global, self.first = K_global, first
        M = np.ones(K_global) if M_global is None else np.asarray(M_global, np.float64)
        self.w = M / M.sum()

    def mean_buffer(self):
        self.mean = torch.zeros(self.P, dtype=torch.float64)
        return self.mean

    def set_params(self, x0):
        self.o.set_params(x0)

    def local_step(self, g):
        self.log.append("step")
        self.o.local_step(g)

    def comm_begin(self, side):
        assert self.phase == "idle"
        self.log.append("begin")
        self.o.snap[:] = self.o.x
        if self.attached is None:
            w = self.w[self.first:self.first + self.K]
            self.mean.copy_(torch.from_numpy((w[:, None] * self.o.snap.astype(np.float64)).sum(0)))
            self.phase = "started"
        else:
            self.phase = "begun"

    def ipc_export(self):
        return ("blob", self.first, self.K)

    def ipc_attach(self, rank, blobs):
        assert [b[0] for b in blobs] == ["blob"] * len(blobs) and blobs[rank] == self.ipc_export()
        assert [b[1] for b in blobs] == list(np.cumsum([0] + [b[2] for b in blobs[:-1]]))
        self.attached = (rank, len(blobs))

    def comm_gather(self):
        assert self.phase == "begun"
        self.log.append("gather")
        rank, G = self.attached
        snaps = [None] * G
        dist.all_gather_object(snaps, self.o.snap)               # stands in for the peer loads
        allsnap = np.concatenate(snaps, 0).astype(np.float64)
        lo, hi = self.P * rank // G, self.P * (rank + 1) // G     # this process's share of the columns
        mine = (self.w[:, None] * allsnap[:, lo:hi]).sum(0)
        parts = [None] * G
        dist.all_gather_object(parts, mine)                       # stands in for the peer stores
        self.mean.copy_(torch.from_numpy(np.concatenate(parts)))
        self.phase = "started"

    def comm_exchanged(self):
        assert self.phase == "started"
        self.log.append("exchanged")
        self.o.mean[:] = self.mean.numpy().astype(np.float32)
        self.o.in_flight = True
        self.phase = "complete"

    def comm_end(self):
        assert self.phase == "complete"
        self.log.append("end")
        self.o.comm_end()
        self.phase = "idle"

    def get_params(self, out=None):
        return self.o.x

    def sync(self):
        pass

    def ipc_detach(self):
        self.attached = None

    def destroy(self):
        pass


def _worker(rank, world, port, K_global, M, exchange, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    eng = WorkerShardedEngine(K_global, P, LR, MU, WD, batch_sizes=M, exchange=exchange, sync="host",
                              engine_factory=HostEngine)
    first, count = shard_workers(K_global, world, rank)
    assert (eng.first, eng.K) == (first, count)
    eng.set_params(I.initial_point(P))
    for r in range(ROUNDS):
        eng.comm_begin(None)
        for s in range(k):
            eng.local_step(I.gradients(K_global, P, r * k + s)[first:first + count])
        eng.comm_end()
    np.save(os.path.join(out_dir, f"x{rank}.npy"), eng.get_params())
    log = eng.engine.log
    eng.close()
    per_round = ["begin"] + (["gather"] if exchange == "gather" else []) + ["exchanged"] + ["step"] * k + ["end"]
    assert log == per_round * ROUNDS
    dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("K_global,M,exchange", [
    (4, None, "allreduce"),
    (5, None, "allreduce"),                       # unequal blocks: 3 + 2 workers
    (5, [32, 64, 128, 32, 256], "allreduce"),     # Section 3.2: mini-batch sizes proportional to speed
    (5, [32, 64, 128, 32, 256], "gather"),
    (4, None, "gather"),
])
def test_two_processes_reproduce_algorithm_1_over_all_workers(tmp_path, K_global, M, exchange):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), K_global, M, exchange, str(tmp_path)), nprocs=world, join=True)
    whole = OracleEngine(K_global, P, LR, MU, WD, mode="ref", batch_sizes=M)
    whole.set_params(I.initial_point(P))
    whole.run(lambda t: I.gradients(K_global, P, t), k, ROUNDS)
    got = np.concatenate([np.load(tmp_path / f"x{r}.npy") for r in range(world)], axis=0)
    assert got.shape == whole.x.shape
    # the spread changes only the order of an fp64 sum: at most the last bit of a few elements
    np.testing.assert_allclose(got, whole.x, rtol=2e-7, atol=1e-9)
    assert np.mean(got.view(np.uint32) == whole.x.view(np.uint32)) > 0.999


def test_shard_workers_tiles_the_workers():
    for K_global in (1, 2, 5, 16, 17, 64):
        for G in range(1, min(K_global, 9) + 1):
            blocks = [shard_workers(K_global, G, r) for r in range(G)]
            assert blocks[0][0] == 0 and sum(c for _, c in blocks) == K_global
            assert all(blocks[r + 1][0] == blocks[r][0] + blocks[r][1] for r in range(G - 1))
            sizes = [c for _, c in blocks]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        shard_workers(2, 3, 0)
