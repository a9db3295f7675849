"""The synthetic workloads (sizes and hyper-parameters only; no arithmetic).

The paper trains ResNet18 and VGG16 on CIFAR with 16 workers (Section 5.1); the engine's cost
depends only on K, P, k, so flattened Gaussian vectors of those models' sizes stand in for them.
Fields: K workers, P parameters per worker, k local steps per round, rounds, lr, mu, wd.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class Workload:
    name: str
    K: int
    P: int
    k: int
    rounds: int
    lr: float
    mu: float
    wd: float
    sigma_x0: float = 0.01
    sigma_g: float = 0.01

    @property
    def n(self) -> int:
        return self.K * self.P

    def bytes_per_round(self, snapshot_copy: bool = False) -> int:
        """Algorithmic HBM bytes of one round: k local steps (20 B per worker-parameter), the
        stored copy (8 B, or 0 with the buffer flip), the mean (4 B + 4 B / K) and the merge
        (12 B + 4 B / K)."""
        per_wp = 20 * self.k + (8 if snapshot_copy else 0) + 4 + 12
        return per_wp * self.n + 8 * self.P


WORKLOADS = {
    "tiny": Workload("tiny", K=4, P=100_000, k=4, rounds=10, lr=0.1, mu=0.9, wd=5e-4),
    "resnet18": Workload("resnet18", K=16, P=11_689_512, k=2, rounds=50, lr=0.1, mu=0.9, wd=5e-4),
    "vgg16": Workload("vgg16", K=16, P=138_357_544, k=4, rounds=20, lr=0.05, mu=0.9, wd=5e-4),
}

# algorithmic bytes per worker-parameter of each kernel (fp32)
BYTES_LOCAL_STEP = 20          # read g, x, v ; write x, v
BYTES_SNAPSHOT = 8             # read x ; write stored copy


def bytes_mean(K: int) -> float:
    return 4.0 * (1.0 + 1.0 / K)      # read K stored copies, write one average


def bytes_merge(K: int) -> float:
    return 12.0 + 4.0 / K             # read x, stored copy (+ average once per column) ; write x


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per worker-parameter measured by one
# `ncu --set full` capture of these three kernels on a small case (K=16, P=4,194,304); pure
# streaming, so it scales with K*P.
NCU_DRAM_BYTES_PER_WORKER_PARAM = {"local_step": 19.25, "mean": 4.12, "merge": 11.81}

# The same for one launch of the persistent gradient + update kernel of the end-to-end MLP workload (K = 16 workers,
# 784-1024-1024-10): dram__bytes_read.sum + dram__bytes_write.sum of one `ncu --set full` capture, in bytes.  (Below the
# 533 MB it moves algorithmically because the tail of its output is still in L2 when it ends.)
NCU_DRAM_BYTES_MLP_UPDATE_KERNEL_K16 = 252.9e6 + 242.0e6
