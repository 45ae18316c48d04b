"""Helpers shared by the tests: build the CPU checker and the CUDA network for
one workload from the same seeded fp32 inputs, and compare them."""
from __future__ import annotations

import numpy as np

from paper_2008_01425_b200 import workloads as wl

PARITY_LINES = []     # one line per parity run, printed by conftest.py after the test summary


def oracle_for(w: wl.Workload):
    from oracle import pg_oracle as po

    return po.Oracle(kind=w.kind, n_workers=w.n_workers, layer_shapes=w.layer_shapes, rank=w.rank,
                     power_steps=w.power_steps, seed=w.seed, torus_rows=w.torus_rows,
                     torus_cols=w.torus_cols, custom_edges=w.custom_edges,
                     weight_rule=w.weight_rule, W=wl.mixing_matrix(w))


def network_for(w: wl.Workload, device: str = "cuda:0"):
    from paper_2008_01425_b200 import binding as pg

    return pg.PowerGossip(kind=w.kind, n_workers=w.n_workers, layer_shapes=w.layer_shapes, rank=w.rank,
                          power_steps=w.power_steps, seed=w.seed, torus_rows=w.torus_rows,
                          torus_cols=w.torus_cols, custom_edges=w.custom_edges,
                          weight_rule=w.weight_rule, W=wl.mixing_matrix(w), device=device)


def load_both(w: wl.Workload, oracle, net) -> None:
    """Same seeded fp32 X^(0) into both sides, one matrix at a time."""
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            x = wl.initial_params(w, i, l)
            if oracle is not None:
                oracle.set_params(i, l, x)
            if net is not None:
                net.pg_write_params(i, l, x)


FP32_FLOOR = 5e-7     # an error of this part of ||X|| is a few units in the last place of the fp32 values X is stored in


def relative_errors(w: wl.Workload, oracle, net, x0=None):
    """Two figures per (worker, layer), each returned as (maximum, where):

    on_x        ||X_gpu - X_oracle||_F / ||X_oracle||_F, the tolerance figure;
    on_change   ||X_gpu - X_oracle||_F / ||X_oracle - X0||_F, the same error against
                what the rounds have changed since X0 (the seeded initial matrices,
                or the caller's `x0[worker][layer]`, e.g. the state of the last
                re-basing).  On stacks whose workers share a large common part this
                is the stricter figure, because one round moves only a small part of ||X||.
                Matrices whose on_x is below FP32_FLOOR are left out of this maximum:
                their error is already at the resolution X is stored with, and once
                the workers nearly agree a few rounds change less than that.
    """
    on_x, on_change = (0.0, None), (0.0, None)
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            ref = oracle.get_params(i, l)
            got = net.pg_read_params(i, l).astype(np.float64)
            start = wl.initial_params(w, i, l) if x0 is None else x0[i][l]
            diff = np.linalg.norm(got - ref)
            a = diff / max(np.linalg.norm(ref), 1e-300)
            moved = np.linalg.norm(ref - start)
            b = diff / moved if moved > 0.0 else (0.0 if diff == 0.0 else np.inf)
            if not np.isfinite(a) or a > on_x[0]:
                on_x = (float(a), (i, l))
            if a > FP32_FLOOR and (not np.isfinite(b) or b > on_change[0]):
                on_change = (float(b), (i, l))
    return on_x, on_change


def max_relative_error(w: wl.Workload, oracle, net):
    """max over (worker, layer) of ||X_gpu - X_oracle||_F / ||X_oracle||_F, and where."""
    worst = 0.0
    where = None
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            ref = oracle.get_params(i, l)
            got = net.pg_read_params(i, l).astype(np.float64)
            err = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
            if not np.isfinite(err) or err > worst:
                worst, where = float(err), (i, l)
    return worst, where


def gpu_average(w: wl.Workload, net, layer: int) -> np.ndarray:
    acc = np.zeros(w.layer_shapes[layer], dtype=np.float64)
    for i in range(w.n_workers):
        acc += net.pg_read_params(i, layer)
    return acc / w.n_workers


def initial_average(w: wl.Workload, layer: int) -> np.ndarray:
    acc = np.zeros(w.layer_shapes[layer], dtype=np.float64)
    for i in range(w.n_workers):
        acc += wl.initial_params(w, i, layer)
    return acc / w.n_workers


def rebase(w: wl.Workload, oracle, net, pairs) -> None:
    """Round the checker's own state to fp32 and load those bits into both sides.

    Data only flows from the checker to the CUDA path.  After this call both
    hold identical fp32 parameters and per-pair vectors; `pairs` lists the
    pairs whose vectors have been touched so far.  Returns the loaded matrices,
    [worker][layer], the state the next segment starts from.
    """
    loaded = []
    for i in range(w.n_workers):
        row = []
        for l in range(len(w.layer_shapes)):
            x32 = oracle.get_params(i, l).astype(np.float32)
            oracle.set_params(i, l, x32)
            net.pg_write_params(i, l, x32)
            row.append(x32)
        loaded.append(row)
    for (i, j) in sorted(pairs):
        for l in range(len(w.layer_shapes)):
            q32 = oracle.get_q(i, j, l).astype(np.float32)
            oracle.set_q(i, j, l, q32.astype(np.float64))
            net.pg_write_q(i, j, l, q32)
    return loaded


def gpu_consensus_distance(w: wl.Workload, net) -> float:
    """(1/N) sum_i ||X_i - mean_j X_j||_F^2 over all layers, from the GPU's parameters."""
    total = 0.0
    for l in range(len(w.layer_shapes)):
        xs = [net.pg_read_params(i, l).astype(np.float64) for i in range(w.n_workers)]
        mean = sum(xs) / w.n_workers
        total += sum(float(np.sum((x - mean) ** 2)) for x in xs)
    return total / w.n_workers
