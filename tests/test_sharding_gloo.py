"""The N > 1 path on CPU (gloo, world_size 2): the parameter path shards by column with no
exchange, so two ranks that each run Algorithm 1 on their own column range must reproduce, bit
for bit, the matching slices of one run over the whole vector; the only collective is the
max-over-ranks of the timed region."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle.cocod_oracle import OracleEngine
from paper_1906_12043_b200 import inputs as I

K, P, k, ROUNDS = 3, 1000, 2, 3
LR, MU, WD = 0.1, 0.9, 5e-4


def run_columns(p0, n):
    cols = np.arange(p0, p0 + n, dtype=np.uint64)
    eng = OracleEngine(K, n, LR, MU, WD, mode="ref")
    eng.set_params(I.initial_point(0, cols=cols))
    eng.run(lambda t: I.gradients(K, 0, t, cols=cols), k, ROUNDS)
    return eng.x.copy()


def _worker(rank, world, port, weak, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    if weak:                              # bench.py's layout: every rank owns P columns of an N*P vector
        lo, hi = rank * P, (rank + 1) * P
    else:                                 # strong: one vector of P columns split by shard_columns
        lo, hi = I.shard_columns(P, rank, world)
    x = run_columns(lo, hi - lo)
    np.save(os.path.join(out_dir, f"x{rank}.npy"), x)
    ms = torch.tensor([10.0 + rank], dtype=torch.float64)       # stands in for this rank's timed region
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    np.save(os.path.join(out_dir, f"t{rank}.npy"), ms.numpy())
    dist.barrier()
    dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("weak", [True, False])
def test_two_ranks_reproduce_the_unsharded_run(tmp_path, weak):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), weak, str(tmp_path)), nprocs=world, join=True)
    total = world * P if weak else P
    whole = run_columns(0, total)
    got = np.concatenate([np.load(tmp_path / f"x{r}.npy") for r in range(world)], axis=1)
    assert got.shape == whole.shape
    np.testing.assert_array_equal(got.view(np.uint32), whole.view(np.uint32))
    for r in range(world):                # every rank sees the slowest rank's time
        assert np.load(tmp_path / f"t{r}.npy")[0] == 10.0 + world - 1
