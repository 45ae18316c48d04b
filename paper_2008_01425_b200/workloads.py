"""Seeded synthetic workloads: shapes, topologies and initial parameter stacks.

This module holds no PowerGossip arithmetic.  It only describes the five
workloads (who is connected to whom is left to the schedule builders; here a
topology is just a kind plus its integer dimensions) and draws the initial
fp32 parameter matrices X_i[l] with numpy's counter-seeded generators, so that
the CPU checker and the CUDA library can be fed the very same bits.

The shapes stand in for the models the paper trains: the ResNet-20 matrix
shapes are those of the paper's ResNet-20 parameter table (Appendix
"Network architectures"), the LSTM stack follows the paper's LSTM parameter
table with the vocabulary rounded to 28000 and a separate decoder, and the
VGG-16 stack is the CIFAR variant with three small fully connected layers.
No dataset item or trained weight is used anywhere: every value is drawn from
the stated distribution.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

# Topology kinds (plain integers shared by both C interfaces).
RING = 0
TORUS = 1
MATCHING = 2
CUSTOM = 3

# Weight rules.
W_UNIFORM = 0      # 1 / (max_degree + 1) on every edge
W_METROPOLIS = 1   # 1 / (1 + max(deg_i, deg_j))
W_EXPLICIT = 2     # caller supplies the N x N mixing matrix


@dataclass(frozen=True)
class Workload:
    """One synthetic PowerGossip workload."""

    name: str
    config_id: int
    n_workers: int
    kind: int
    torus_rows: int
    torus_cols: int
    weight_rule: int
    neighbour_weight: Optional[float]   # explicit ring weight, else None
    layer_shapes: Tuple[Tuple[int, int], ...]
    rank: int
    power_steps: int
    rounds: int
    seed: int
    init: str                           # recipe name, see initial_params()
    custom_edges: Tuple[Tuple[int, int], ...] = field(default=())

    @property
    def params_per_worker(self) -> int:
        return int(sum(n * m for n, m in self.layer_shapes))

    @property
    def total_params(self) -> int:
        return self.params_per_worker * self.n_workers

    def replace(self, **kw) -> "Workload":
        d = dict(self.__dict__)
        d.update(kw)
        return Workload(**d)


RESNET20_SHAPES: Tuple[Tuple[int, int], ...] = (
    ((16, 27),)
    + ((16, 144),) * 6
    + ((32, 144),)
    + ((32, 288),) * 5
    + ((32, 16),)
    + ((64, 288),)
    + ((64, 576),) * 5
    + ((64, 32),)
    + ((10, 64),)
)

VGG16_SHAPES: Tuple[Tuple[int, int], ...] = (
    (64, 27), (64, 576), (128, 576), (128, 1152), (256, 1152),
    (256, 2304), (256, 2304), (512, 2304),
    (512, 4608), (512, 4608), (512, 4608), (512, 4608), (512, 4608),
    (512, 512), (512, 512), (10, 512),
)

LSTM_SHAPES: Tuple[Tuple[int, int], ...] = (
    ((28000, 650),) + ((2600, 650),) * 6 + ((650, 28000),)
)


def tiny_ring() -> Workload:
    return Workload("tiny_ring4_64x32", 1, 4, RING, 0, 0, W_EXPLICIT, 1.0 / 3.0,
                    ((64, 32),), 1, 1, 20, 1001, "normal1")


def resnet20_ring8() -> Workload:
    return Workload("resnet20_ring8", 2, 8, RING, 0, 0, W_EXPLICIT, 0.436,
                    RESNET20_SHAPES, 1, 1, 100, 1002, "normal0.05")


def torus8x8(power_steps: int = 1, rounds: int = 200) -> Workload:
    return Workload("torus8x8_1024sq_P%d" % power_steps, 3, 64, TORUS, 8, 8,
                    W_METROPOLIS, None, ((1024, 1024),), 1, power_steps, rounds,
                    1003, "normal1_plus_rank4")


def vgg16_ring16(rank: int = 1) -> Workload:
    return Workload("vgg16_ring16_r%d" % rank, 4, 16, RING, 0, 0, W_EXPLICIT,
                    1.0 / 3.0, VGG16_SHAPES, rank, 2, 50, 1004,
                    "shared0.02_plus0.002")


def lstm_matching32() -> Workload:
    return Workload("lstm_matching32", 5, 32, MATCHING, 0, 0, W_METROPOLIS, None,
                    LSTM_SHAPES, 1, 1, 20, 1005, "uniform0.1")


def consensus_ring8(iterations_per_round: int = 1, rounds: int = 400) -> Workload:
    """The paper's consensus experiment (Appendix "Experimental settings", table
    "Experimental settings for Consensus"): 8 workers in a ring, one 100 x 100
    standard-normal matrix each, W = 0.436 / 0.128."""
    return Workload("consensus_ring8_100x100", 6, 8, RING, 0, 0, W_EXPLICIT, 0.436,
                    ((100, 100),), 1, iterations_per_round, rounds, 1006, "normal1")


def all_workloads() -> List[Workload]:
    return [tiny_ring(), resnet20_ring8(), torus8x8(1), torus8x8(2), torus8x8(4),
            vgg16_ring16(1), vgg16_ring16(2), lstm_matching32(), consensus_ring8()]


def by_name(name: str) -> Workload:
    for w in all_workloads():
        if w.name == name:
            return w
    raise KeyError(name)


def shrink(w: Workload, layer_shapes: Sequence[Tuple[int, int]], rounds: int,
           name_suffix: str = "_small") -> Workload:
    """Same recipe on smaller matrices (for cases a CPU checker finishes fast)."""
    return w.replace(name=w.name + name_suffix,
                     layer_shapes=tuple((int(a), int(b)) for a, b in layer_shapes),
                     rounds=int(rounds))


def _rng(w: Workload, worker: int, layer: int, stream: int) -> np.random.Generator:
    return np.random.default_rng([w.config_id, w.seed, worker, layer, stream])


def initial_params(w: Workload, worker: int, layer: int) -> np.ndarray:
    """fp32 X_worker[layer] at round 0, dense row-major (rows x cols)."""
    n, m = w.layer_shapes[layer]
    g = _rng(w, worker, layer, 0)
    if w.init == "normal1":
        x = g.standard_normal((n, m), dtype=np.float32)
    elif w.init == "normal0.05":
        x = g.standard_normal((n, m), dtype=np.float32) * np.float32(0.05)
    elif w.init == "normal1_plus_rank4":
        x = g.standard_normal((n, m), dtype=np.float32)
        k = min(4, n, m)
        u = g.standard_normal((n, k), dtype=np.float32)
        v = g.standard_normal((m, k), dtype=np.float32)
        scale = (0.5 ** np.arange(k)).astype(np.float32)
        x = x + (u * scale) @ v.T
    elif w.init == "shared0.02_plus0.002":
        shared = np.random.default_rng([w.config_id, w.seed, 1 << 20, layer, 1])
        base = shared.standard_normal((n, m), dtype=np.float32) * np.float32(0.02)
        x = base + g.standard_normal((n, m), dtype=np.float32) * np.float32(0.002)
    elif w.init == "uniform0.1":
        x = (g.random((n, m), dtype=np.float32) - np.float32(0.5)) * np.float32(0.2)
    else:
        raise ValueError("unknown init recipe %r" % (w.init,))
    return np.ascontiguousarray(x, dtype=np.float32)


def mixing_matrix(w: Workload) -> Optional[np.ndarray]:
    """The explicit N x N fp32 mixing matrix for ring workloads that fix one.

    Returns None when the weight rule is computed by the schedule builder
    (Metropolis-Hastings / uniform).  Only the ring layout is known here; the
    entries are constants copied from the workload description, not computed
    from the method.
    """
    if w.weight_rule != W_EXPLICIT:
        return None
    assert w.kind == RING
    N = w.n_workers
    a = np.float32(w.neighbour_weight)
    W = np.zeros((N, N), dtype=np.float32)
    for i in range(N):
        for j in ((i + 1) % N, (i - 1) % N):
            if j != i:
                W[i, j] = a
    for i in range(N):
        W[i, i] = np.float32(1.0) - W[i].sum(dtype=np.float32)
    return W
