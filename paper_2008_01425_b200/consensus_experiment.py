"""The paper's consensus experiment on the GPU library.

Eight workers in a ring start from unrelated 100 x 100 standard-normal matrices
and run compressed gossip only (no gradients).  Reported, as in the paper's
consensus figure: the consensus error (1/8) sum_i ||X_i - mean(X^(0))||_F^2 against
the number of floats every worker has sent to each neighbour.  PowerGossip runs
in the paper-literal mode (Algorithm 2, one iteration per gossip step: 100 floats
per step per neighbour); plain gossip sends the whole matrix (10 000 floats per
step) and follows X <- W X.

    python -m paper_2008_01425_b200.consensus_experiment [--steps 400] [--every 40]
"""
from __future__ import annotations

import argparse

import numpy as np

from . import binding as pg
from . import workloads as wl


def consensus_error(xs, mean0) -> float:
    return float(sum(np.sum((x.astype(np.float64) - mean0) ** 2) for x in xs) / len(xs))


def powergossip_curve(steps: int, every: int, device: str = "cuda:0"):
    """[(floats sent per neighbour, consensus error)] of PowerGossip, one iteration per step."""
    w = wl.consensus_ring8(1, steps)
    net = pg.PowerGossip(kind=w.kind, n_workers=w.n_workers, layer_shapes=w.layer_shapes, rank=1,
                         power_steps=1, seed=w.seed, weight_rule=w.weight_rule, W=wl.mixing_matrix(w),
                         device=device)
    x0 = [wl.initial_params(w, i, 0) for i in range(w.n_workers)]
    for i, x in enumerate(x0):
        net.pg_write_params(i, 0, x)
    net.pg_set_half_step()
    mean0 = sum(x.astype(np.float64) for x in x0) / w.n_workers
    curve = [(0.0, consensus_error(x0, mean0))]
    sent = 0.0
    ends = 2 * len(net.pg_get_schedule(0)[0])       # every edge has two ends
    for t in range(1, steps + 1):
        # what one worker sends one neighbour in this round: the library's count for all ends, per end
        sent += net.pg_comm_floats_round(t - 1)[0] / ends
        net.pg_round()
        if t % every == 0 or t == steps:
            xs = [net.pg_read_params(i, 0) for i in range(w.n_workers)]
            curve.append((sent, consensus_error(xs, mean0)))
    net.close()
    return curve


def plain_gossip_curve(steps: int):
    """Uncompressed gossip X <- W X on the same start (host arithmetic on 8 small matrices)."""
    w = wl.consensus_ring8()
    X = np.stack([wl.initial_params(w, i, 0).astype(np.float64) for i in range(w.n_workers)])
    W = wl.mixing_matrix(w).astype(np.float64)
    mean0 = X.mean(axis=0)
    n, m = w.layer_shapes[0]
    curve = [(0.0, consensus_error(list(X), mean0))]
    for t in range(1, steps + 1):
        X = np.einsum("ij,jnm->inm", W, X)
        curve.append((float(t * n * m), consensus_error(list(X), mean0)))
    return curve


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--every", type=int, default=40)
    args = ap.parse_args()
    print("PowerGossip (Algorithm 2, 1 iteration per step)")
    for sent, err in powergossip_curve(args.steps, args.every):
        print("  floats sent per neighbour %9.0f   consensus error %.6e" % (sent, err))
    print("plain gossip (full matrices)")
    for sent, err in plain_gossip_curve(4):
        print("  floats sent per neighbour %9.0f   consensus error %.6e" % (sent, err))


if __name__ == "__main__":
    main()
