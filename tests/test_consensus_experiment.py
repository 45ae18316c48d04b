"""The paper's consensus experiment (8-ring, 100 x 100 standard-normal matrices,
W = 0.436 / 0.128) as a second workload."""
import numpy as np
import pytest

from paper_2008_01425_b200 import workloads as wl
from tests import common


def _oracle_curve(steps, every):
    w = wl.consensus_ring8(1, steps)
    o = common.oracle_for(w)
    o.set_half_step()
    common.load_both(w, o, None)
    mean0 = common.initial_average(w, 0)
    out = [float(sum(np.sum((o.get_params(i, 0) - mean0) ** 2) for i in range(8)) / 8)]
    for t in range(1, steps + 1):
        o.round()
        if t % every == 0:
            out.append(float(sum(np.sum((o.get_params(i, 0) - mean0) ** 2) for i in range(8)) / 8))
    o.close()
    return out


def test_consensus_error_falls_monotonically():
    """Compressed gossip only: the error against the conserved initial average never
    grows (the update is a projection) and has fallen 40-fold after 400 iterations
    (4 full matrices' worth of floats)."""
    curve = _oracle_curve(400, 40)
    assert all(b < a for a, b in zip(curve, curve[1:]))
    assert curve[-1] < curve[0] / 30


def test_plain_gossip_contracts_at_the_spectral_rate():
    """The uncompressed reference curve: X <- W X contracts the error by at least
    lambda_2(W)^2 per step (classical consensus rate, Theorem 1 with delta = 1)."""
    from paper_2008_01425_b200.consensus_experiment import plain_gossip_curve

    W = wl.mixing_matrix(wl.consensus_ring8()).astype(np.float64)
    lam = np.sort(np.abs(np.linalg.eigvalsh(W)))[::-1]
    assert abs(lam[0] - 1.0) < 1e-6
    plain = plain_gossip_curve(6)
    for (_, a), (_, b) in zip(plain, plain[1:]):
        assert b <= lam[1] ** 2 * a * (1 + 1e-9)
    assert plain[1][0] == 100 * 100


@pytest.mark.gpu
def test_gpu_curve_matches_the_checker():
    from paper_2008_01425_b200.consensus_experiment import powergossip_curve

    gpu = powergossip_curve(200, 20)
    ref = _oracle_curve(200, 20)
    assert len(gpu) == len(ref)
    assert gpu[-1][0] == 200 * 100
    for (sent, e_gpu), e_ref in zip(gpu, ref):
        assert abs(e_gpu - e_ref) <= 0.02 * e_ref, (sent, e_gpu, e_ref)
