"""Pins for the fp64 CPU checker: what the paper and the mathematics fix.

None of these compares the checker with itself or with the CUDA path.  Each
test states which passage of the paper (or which textbook fact) it rests on.
"""
import os

import numpy as np
import pytest

from oracle import pg_oracle as po

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def _fill(o, rng, scale=1.0):
    xs = []
    for i in range(o.n_workers):
        row = []
        for l, (n, m) in enumerate(o.layer_shapes):
            x = (rng.standard_normal((n, m)) * scale).astype(np.float32)
            o.set_params(i, l, x)
            row.append(x.astype(np.float64))
        xs.append(row)
    return xs


def _ring_W(N, a):
    W = np.zeros((N, N), dtype=np.float32)
    for i in range(N):
        for j in ((i + 1) % N, (i - 1) % N):
            if j != i:
                W[i, j] = a
    for i in range(N):
        W[i, i] = 1.0 - W[i].sum()
    return W


# --------------------------------------------------------------------------
# random numbers and schedules
# --------------------------------------------------------------------------
def test_philox_known_answers():
    """Philox4x32-10 against the published known-answer vectors."""
    for row in _golden_rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in row]
        assert po.philox4x32_10(v[:4], v[4:6]) == tuple(v[6:])


def test_init_q_is_standard_normal_and_keyed():
    """Algorithm 2 initialises every entry from a standard normal."""
    q = po.init_q(7, 0, 1, 0, 0, 200000).astype(np.float64)
    assert abs(q.mean()) < 0.01
    assert abs(q.std() - 1.0) < 0.01
    assert abs((q ** 3).mean()) < 0.03           # skewness 0
    assert abs((q ** 4).mean() - 3.0) < 0.08     # kurtosis 3
    # a prefix of a longer draw is the shorter draw; any key change gives new numbers
    assert np.array_equal(po.init_q(7, 0, 1, 0, 0, 37), q[:37].astype(np.float32))
    for other in (po.init_q(8, 0, 1, 0, 0, 64), po.init_q(7, 0, 2, 0, 0, 64),
                  po.init_q(7, 1, 2, 0, 0, 64), po.init_q(7, 0, 1, 1, 0, 64),
                  po.init_q(7, 0, 1, 0, 1, 64)):
        assert not np.array_equal(other, q[:64].astype(np.float32))


def test_ring_and_torus_schedules():
    """Ring: N edges, degree 2.  Torus RxC: 2N edges, degree 4, symmetric."""
    for N in (3, 4, 8, 16):
        e = po.schedule(po.RING, N)
        assert len(e) == N
        assert np.all(e[:, 0] < e[:, 1])
        deg = np.bincount(e.ravel(), minlength=N)
        assert np.all(deg == 2)
        assert [tuple(x) for x in e] == sorted(set(tuple(x) for x in e))
        for a, b in e:
            assert (b - a) % N in (1, N - 1)
    assert [tuple(x) for x in po.schedule(po.RING, 2)] == [(0, 1)]
    e = po.schedule(po.TORUS, 64, 8, 8)
    assert len(e) == 128
    assert np.all(np.bincount(e.ravel(), minlength=64) == 4)
    for a, b in e:
        ra, ca, rb, cb = a // 8, a % 8, b // 8, b % 8
        assert ((ra == rb and (ca - cb) % 8 in (1, 7)) or (ca == cb and (ra - rb) % 8 in (1, 7)))
    # a 2x4 torus has doubled vertical links: they are merged
    e = po.schedule(po.TORUS, 8, 2, 4)
    assert len(e) == 8 + 4
    with pytest.raises(ValueError):
        po.schedule(po.TORUS, 10, 3, 3)


def test_matching_schedule():
    """Time-varying graph: a perfect matching drawn afresh every round."""
    N = 32
    seen = set()
    for t in range(50):
        e = po.schedule(po.MATCHING, N, seed=5, round_index=t)
        assert len(e) == N // 2
        assert sorted(e.ravel().tolist()) == list(range(N))
        assert np.all(e[:, 0] < e[:, 1])
        assert list(e[:, 0]) == sorted(e[:, 0])
        assert np.array_equal(e, po.schedule(po.MATCHING, N, seed=5, round_index=t))
        seen.add(tuple(map(tuple, e)))
    assert len(seen) == 50
    assert not np.array_equal(po.schedule(po.MATCHING, N, seed=6, round_index=0),
                              po.schedule(po.MATCHING, N, seed=5, round_index=0))
    with pytest.raises(ValueError):
        po.schedule(po.MATCHING, 7)
    # every pair is about equally likely to be matched: N-1 = 31 possible partners
    hits = np.zeros((8, 8))
    T = 7000
    for t in range(T):
        for a, b in po.schedule(po.MATCHING, 8, seed=11, round_index=t):
            hits[a, b] += 1
    freq = hits[np.triu_indices(8, 1)] / T
    assert np.all(np.abs(freq - 1.0 / 7.0) < 0.02)


def test_mixing_weights_satisfy_A4():
    """Assumption A4: W symmetric, doubly stochastic, non-zero only on edges."""
    for row in _golden_rows("mixing_presets.txt"):
        N, a, s = int(row[0]), float(row[1]), float(row[2])
        assert abs(2 * a + s - 1.0) < 1e-12          # the printed constants are a valid row
        e = po.schedule(po.RING, N)
        w = po.edge_weights(po.W_EXPLICIT, N, e, _ring_W(N, a))
        assert np.allclose(w, a, atol=1e-7)
    e = po.schedule(po.TORUS, 64, 8, 8)
    assert np.allclose(po.edge_weights(po.W_METROPOLIS, 64, e), 1.0 / 5.0)
    assert np.allclose(po.edge_weights(po.W_UNIFORM, 4, po.schedule(po.RING, 4)), 1.0 / 3.0)
    # a star graph: Metropolis weights 1/(1+max degree of the two ends)
    star = np.array([[0, 1], [0, 2], [0, 3]], dtype=np.int32)
    assert np.allclose(po.edge_weights(po.W_METROPOLIS, 4, star), 0.25)
    bad = _ring_W(4, 1.0 / 3.0)
    bad[0, 1] = 0.5                                   # not symmetric, row sum off
    with pytest.raises(ValueError):
        po.edge_weights(po.W_EXPLICIT, 4, po.schedule(po.RING, 4), bad)
    bad = _ring_W(4, 1.0 / 3.0)
    bad[0, 2] = bad[2, 0] = 0.1                       # weight on a non-edge
    bad[0, 0] -= 0.1
    bad[2, 2] -= 0.1
    with pytest.raises(ValueError):
        po.edge_weights(po.W_EXPLICIT, 4, po.schedule(po.RING, 4), bad)


def test_compression_ratios_printed_in_the_paper():
    """Per-tensor ratios of the ResNet-20 and LSTM parameter tables: one
    iteration of Algorithm 2 moves (rows + cols)/2 floats on average."""
    for n, m, printed in _golden_rows("compression_ratios.txt"):
        n, m, printed = int(n), int(m), int(printed)
        assert round(po.compression_ratio(n, m, 1, 1)) == printed
        assert abs(po.compression_ratio(n, m, 1, 4) * 4 - po.compression_ratio(n, m, 1, 1)) < 1e-9


# --------------------------------------------------------------------------
# the gossip round
# --------------------------------------------------------------------------
CASES = [
    dict(kind=po.RING, n_workers=4, layer_shapes=[(9, 7)], rank=1, power_steps=1,
         weight_rule=po.W_EXPLICIT, W=_ring_W(4, 1.0 / 3.0)),
    dict(kind=po.RING, n_workers=8, layer_shapes=[(6, 11), (5, 3)], rank=1, power_steps=2,
         weight_rule=po.W_EXPLICIT, W=_ring_W(8, 0.436)),
    dict(kind=po.TORUS, n_workers=12, torus_rows=3, torus_cols=4, layer_shapes=[(10, 8)],
         rank=2, power_steps=2, weight_rule=po.W_METROPOLIS),
    dict(kind=po.MATCHING, n_workers=6, layer_shapes=[(7, 12), (4, 4)], rank=1, power_steps=1),
    dict(kind=po.MATCHING, n_workers=6, layer_shapes=[(7, 12)], rank=3, power_steps=2),
    dict(kind=po.CUSTOM, n_workers=5, custom_edges=[(0, 1), (0, 2), (0, 3), (3, 4)],
         layer_shapes=[(8, 8)], rank=1, power_steps=1, weight_rule=po.W_METROPOLIS),
]


@pytest.mark.parametrize("case", CASES)
def test_average_is_conserved_and_distance_never_grows(case):
    """Lemma 1 (every edge adds to i what it takes from j, so the worker average
    never moves), and the consensus distance sum_i ||X_i - mean||^2 cannot grow
    in a step: with projectors Pi_e the update is Delta <- (I - M) Delta with
    0 <= M = sum_e W_e (e_i-e_j)(e_i-e_j)^T (x) Pi_e <= I - W < 2I."""
    rng = np.random.default_rng(3)
    o = po.Oracle(seed=17, **case)
    _fill(o, rng)
    avg0 = [o.average(l) for l in range(len(o.layer_shapes))]
    d_prev = o.consensus_distance()
    for _ in range(12):
        o.round()
        for l in range(len(o.layer_shapes)):
            scale = np.abs(avg0[l]).max()
            assert np.abs(o.average(l) - avg0[l]).max() <= 1e-13 * max(scale, 1.0)
        d = o.consensus_distance()
        assert d <= d_prev * (1 + 1e-12)
        d_prev = d
    assert np.isfinite(d_prev)
    o.close()


def test_rank1_difference_is_removed_exactly():
    """If X_i - X_j = sigma u v^T, then C_v recovers it exactly (Section 4: with v
    the top right singular vector C_v(X) is the best rank-1 approximation, here
    exact): p ~ u, q' = D^T u = sigma v, so the step equals uncompressed gossip on
    that edge; with W_ij = 1/2 both workers land on their average at once."""
    rng = np.random.default_rng(5)
    n, m = 12, 9
    base = rng.standard_normal((n, m)).astype(np.float32)
    u = rng.standard_normal((n, 1)).astype(np.float32)
    v = rng.standard_normal((1, m)).astype(np.float32)
    # pick entries that are exact in fp32 so that the difference is exactly rank 1
    base = np.round(base * 64) / 64
    u = np.round(u * 8) / 8
    v = np.round(v * 8) / 8
    x0 = (base + u @ v).astype(np.float32)
    x1 = base.astype(np.float32)
    for w_edge in (0.5, 0.3):
        W = np.array([[1 - w_edge, w_edge], [w_edge, 1 - w_edge]], dtype=np.float32)
        o = po.Oracle(kind=po.CUSTOM, n_workers=2, custom_edges=[(0, 1)], layer_shapes=[(n, m)],
                      rank=1, power_steps=1, seed=3, weight_rule=po.W_EXPLICIT, W=W)
        o.set_params(0, 0, x0)
        o.set_params(1, 0, x1)
        o.round()
        D0 = x0.astype(np.float64) - x1.astype(np.float64)
        w64 = float(np.float32(w_edge))
        assert np.allclose(o.get_params(0, 0), x0 - w64 * D0, rtol=0, atol=1e-13)
        assert np.allclose(o.get_params(1, 0), x1 + w64 * D0, rtol=0, atol=1e-13)
        if w_edge == 0.5:
            assert np.allclose(o.get_params(0, 0), o.get_params(1, 0), rtol=0, atol=1e-13)
        # the stored vector is now D^T p_hat = +- sigma v
        q = o.get_q(0, 1, 0)[:, 0]
        sigma = np.linalg.norm(u.astype(np.float64)) * np.linalg.norm(v.astype(np.float64))
        assert abs(np.linalg.norm(q) - sigma) < 1e-12 * sigma
        o.close()


@pytest.mark.parametrize("rank", [1, 2, 3])
def test_frozen_difference_converges_to_svd(rank):
    """Eq. 3: on a difference that does not change the scheme is power iteration,
    so the warm-started factors converge to the top singular triplets of
    D = X_0 - X_1 (numpy.linalg.svd), at the rate (sigma_{r+1}/sigma_r)^2 per step.
    The edge weight 0 freezes X."""
    rng = np.random.default_rng(11)
    n, m = 8, 6
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    V, _ = np.linalg.qr(rng.standard_normal((m, m)))
    s = np.array([5.0, 3.0, 1.5, 0.6, 0.2, 0.05])
    D = (U[:, :m] * s) @ V.T
    x1 = rng.standard_normal((n, m)).astype(np.float32)
    x0 = (x1 + D).astype(np.float32)
    Dq = x0.astype(np.float64) - x1.astype(np.float64)          # what the oracle sees
    Us, ss, Vts = np.linalg.svd(Dq)
    W = np.eye(2, dtype=np.float32)
    o = po.Oracle(kind=po.CUSTOM, n_workers=2, custom_edges=[(0, 1)], layer_shapes=[(n, m)],
                  rank=rank, power_steps=1, seed=9, weight_rule=po.W_EXPLICIT, W=W)
    o.set_params(0, 0, x0)
    o.set_params(1, 0, x1)
    proj_true = Us[:, :rank] @ Us[:, :rank].T
    errs = []
    for _ in range(60):
        o.round()
        P = o.get_phat(0, 1, 0)
        errs.append(np.linalg.norm(P @ P.T - proj_true))
    assert np.array_equal(o.get_params(0, 0), x0.astype(np.float64))   # frozen
    P = o.get_phat(0, 1, 0)
    Q = o.get_q(0, 1, 0)
    assert np.allclose(P.T @ P, np.eye(rank), atol=1e-12)             # orthonormal
    assert errs[-1] < 1e-9
    # geometric decay of the subspace error, ratio (s_{r+1}/s_r)^2
    ratio = (ss[rank] / ss[rank - 1]) ** 2
    k0, k1 = 6, 12
    assert errs[k1] / errs[k0] < (ratio ** (k1 - k0)) * 50
    assert errs[k1] / errs[k0] > (ratio ** (k1 - k0)) / 50
    # Q = D^T P: its columns converge to sigma_k v_k (up to sign)
    for k in range(rank):
        assert abs(np.linalg.norm(Q[:, k]) - ss[k]) < 1e-7 * ss[k]
        assert abs(abs(Q[:, k] @ Vts[k]) - ss[k]) < 1e-7 * ss[k]
        assert abs(abs(P[:, k] @ Us[:, k]) - 1.0) < 1e-9
    # P Q^T is the best rank-r approximation of D (Eckart-Young)
    best = (Us[:, :rank] * ss[:rank]) @ Vts[:rank]
    assert np.allclose(P @ Q.T, best, atol=1e-7)
    o.close()


def test_identical_workers_are_a_fixed_point():
    """Section 4.1: if two workers agree their compressed update is zero, so
    consensus is a fixed point; nothing becomes NaN and the stored vectors stay."""
    rng = np.random.default_rng(2)
    x = rng.standard_normal((10, 7)).astype(np.float32)
    o = po.Oracle(kind=po.RING, n_workers=4, layer_shapes=[(10, 7)], rank=2, power_steps=2,
                  seed=4, weight_rule=po.W_EXPLICIT, W=_ring_W(4, 1.0 / 3.0))
    for i in range(4):
        o.set_params(i, 0, x)
    q_before = o.get_q(0, 1, 0)
    o.round(3)
    for i in range(4):
        assert np.array_equal(o.get_params(i, 0), x.astype(np.float64))
    assert np.array_equal(o.get_q(0, 1, 0), q_before)
    o.close()
    # only worker 2 differs: after one power step worker 0, whose two edges carry
    # no difference, has not moved at all
    o = po.Oracle(kind=po.RING, n_workers=4, layer_shapes=[(10, 7)], rank=2, power_steps=1,
                  seed=4, weight_rule=po.W_EXPLICIT, W=_ring_W(4, 1.0 / 3.0))
    for i in range(4):
        o.set_params(i, 0, x)
    y = x.copy()
    y[3, 2] += 1.0
    o.set_params(2, 0, y)
    o.round()
    assert np.array_equal(o.get_params(0, 0), x.astype(np.float64))    # both its edges carry no difference
    for i in (1, 2, 3):
        assert np.all(np.isfinite(o.get_params(i, 0)))
    assert not np.array_equal(o.get_params(1, 0), x.astype(np.float64))
    o.close()


@pytest.mark.parametrize("shape,rank", [((7, 1), 1), ((1, 6), 1), ((3, 5), 3), ((5, 3), 4)])
@pytest.mark.parametrize("topo", ["ring", "torus", "matching"])
def test_full_rank_equals_plain_gossip(shape, rank, topo):
    """With rank >= min(rows, cols) (or a single column / row) the projector
    Ph Ph^T leaves the difference untouched, so one power step is the gossip term
    of D-PSGD (Eq. 1): X <- W X.  Checked against numpy's matrix product."""
    rng = np.random.default_rng(13)
    n, m = shape
    if topo == "ring":
        N = 6
        W = _ring_W(N, 0.3)
        o = po.Oracle(kind=po.RING, n_workers=N, layer_shapes=[shape], rank=rank, power_steps=1,
                      seed=21, weight_rule=po.W_EXPLICIT, W=W)
        W64 = W.astype(np.float64)
    elif topo == "torus":
        N = 12
        o = po.Oracle(kind=po.TORUS, n_workers=N, torus_rows=3, torus_cols=4, layer_shapes=[shape],
                      rank=rank, power_steps=1, seed=21, weight_rule=po.W_METROPOLIS)
        W64 = np.zeros((N, N))
        for a, b in po.schedule(po.TORUS, N, 3, 4):
            W64[a, b] = W64[b, a] = 0.2
        W64 += np.diag(1.0 - W64.sum(1))
    else:
        N = 6
        o = po.Oracle(kind=po.MATCHING, n_workers=N, layer_shapes=[shape], rank=rank,
                      power_steps=1, seed=21)
        W64 = np.zeros((N, N))
        for a, b in po.schedule(po.MATCHING, N, seed=21, round_index=0):
            W64[a, b] = W64[b, a] = 0.5
        W64 += np.diag(1.0 - W64.sum(1))
    xs = _fill(o, rng)
    X = np.stack([xs[i][0] for i in range(N)])            # N x n x m
    o.round()
    expect = np.einsum("ij,jnm->inm", W64, X)
    got = np.stack([o.get_params(i, 0) for i in range(N)])
    assert np.allclose(got, expect, rtol=0, atol=1e-12)
    o.close()


def test_one_step_matches_projector_form():
    """Cross-check of a whole Jacobi step on a ring against the operator form used
    in the proof of Lemma 2: X_i <- X_i + sum_j W_ij Pi_ij (X_j - X_i) with
    Pi_ij = p p^T, p = D q / ||D q||  (numpy, left-projector form)."""
    rng = np.random.default_rng(23)
    N, n, m = 5, 7, 9
    W = _ring_W(N, 0.25)
    o = po.Oracle(kind=po.RING, n_workers=N, layer_shapes=[(n, m)], rank=1, power_steps=1,
                  seed=31, weight_rule=po.W_EXPLICIT, W=W)
    xs = _fill(o, rng)
    X = [xs[i][0] for i in range(N)]
    edges, w = o.round_schedule()
    new = [x.copy() for x in X]
    for (i, j), wij in zip(edges, w):
        q = po.init_q(31, i, j, 0, 0, m).astype(np.float64)
        D = X[i] - X[j]
        p = D @ q
        p /= np.linalg.norm(p)
        Pi = np.outer(p, p)
        new[i] += wij * Pi @ (X[j] - X[i])
        new[j] += wij * Pi @ (X[i] - X[j])
    o.round()
    for i in range(N):
        assert np.allclose(o.get_params(i, 0), new[i], rtol=0, atol=1e-12)
    o.close()


def test_warm_start_is_kept_per_pair_on_a_time_varying_graph():
    """A pair that meets again continues from the vector it stored last time, and
    a pair that has not met yet still has its seed-derived initial vector."""
    N, m = 4, 5
    o = po.Oracle(kind=po.MATCHING, n_workers=N, layer_shapes=[(6, m)], rank=1, power_steps=1, seed=77)
    _fill(o, np.random.default_rng(1))
    met = {}
    for t in range(6):
        edges, _ = o.round_schedule()
        untouched = [(a, b) for a in range(N) for b in range(a + 1, N)
                     if (a, b) not in met and (a, b) not in [tuple(e) for e in edges]]
        o.round()
        for a, b in untouched:
            assert np.array_equal(o.get_q(a, b, 0)[:, 0], po.init_q(77, a, b, 0, 0, m).astype(np.float64))
        for a, b in edges:
            met[(int(a), int(b))] = o.get_q(a, b, 0).copy()
        for (a, b), q in met.items():
            if (a, b) not in [tuple(e) for e in edges]:
                assert np.array_equal(o.get_q(a, b, 0), q)
    o.close()


# --------------------------------------------------------------------------
# rank > 1: columns that depend on earlier ones (Appendix "Changing rank vs
# changing # power iterations" only says "orthogonalized"; the rule for a column
# with nothing left after the projection is this build's reading: it is dropped
# when the squared norm of its residual is at most 1e-10 of its squared norm
# before the projection, i.e. what is left is below 1e-5 of its length)
# --------------------------------------------------------------------------
def _two_workers(n, m, rank, w_edge=0.3, seed=5):
    W = np.array([[1 - w_edge, w_edge], [w_edge, 1 - w_edge]], dtype=np.float32)
    return po.Oracle(kind=po.CUSTOM, n_workers=2, custom_edges=[(0, 1)], layer_shapes=[(n, m)], rank=rank,
                     power_steps=1, seed=seed, weight_rule=po.W_EXPLICIT, W=W)


def _unit_columns(q):
    return q / np.linalg.norm(q, axis=0, keepdims=True)


def test_exactly_dependent_columns_are_dropped_and_keep_their_vector():
    """A column of P that is a combination of earlier columns spans nothing new: it must
    not contribute an update (the projector P-hat P-hat^T is that of the earlier columns
    alone) and its stored vector stays as it was, so that consensus remains a fixed point
    (Section 4.1) and no 0/0 appears.  Two ways to get one: more columns than rows, and a
    repeated column in Q."""
    rng = np.random.default_rng(41)
    # (1) rank 3 on matrices with 2 rows: the third column of P lies in the span of the first two
    n, m = 2, 7
    o = _two_workers(n, m, rank=3)
    xs = _fill(o, rng)
    q_before = o.get_q(0, 1, 0)
    o.round()
    D = xs[0][0] - xs[1][0]
    w64 = float(np.float32(0.3))
    # two independent columns already span R^2: the step is plain gossip on this edge
    assert np.allclose(o.get_params(0, 0), xs[0][0] - w64 * D, rtol=0, atol=1e-13)
    assert np.allclose(o.get_params(1, 0), xs[1][0] + w64 * D, rtol=0, atol=1e-13)
    q_after = o.get_q(0, 1, 0)
    assert np.array_equal(q_after[:, 2], q_before[:, 2])              # dropped column: vector kept
    assert not np.array_equal(q_after[:, 0], q_before[:, 0]) and not np.array_equal(q_after[:, 1], q_before[:, 1])
    P = o.get_phat(0, 1, 0)
    assert np.array_equal(P[:, 2], np.zeros(n))
    assert np.allclose(P[:, :2].T @ P[:, :2], np.eye(2), atol=1e-12)
    assert o.min_residual_ratio() < 1e-24                               # rounding residue only
    o.close()
    # (2) a repeated column: the step is the rank-1 step of the first column
    n, m = 9, 6
    o2 = _two_workers(n, m, rank=2)
    o1 = _two_workers(n, m, rank=1)
    x0 = rng.standard_normal((n, m)).astype(np.float32)
    x1 = rng.standard_normal((n, m)).astype(np.float32)
    for o in (o1, o2):
        o.set_params(0, 0, x0)
        o.set_params(1, 0, x1)
    q = rng.standard_normal((m, 1))
    o1.set_q(0, 1, 0, q)
    o2.set_q(0, 1, 0, np.hstack([q, q]))
    o1.round()
    o2.round()
    for i in range(2):
        assert np.allclose(o2.get_params(i, 0), o1.get_params(i, 0), rtol=0, atol=1e-13)
    assert np.allclose(o2.get_q(0, 1, 0)[:, 0], o1.get_q(0, 1, 0)[:, 0], rtol=0, atol=1e-13)
    assert np.array_equal(o2.get_q(0, 1, 0)[:, 1], q[:, 0])           # kept
    assert np.array_equal(o2.get_phat(0, 1, 0)[:, 1], np.zeros(n))
    o1.close()
    o2.close()


@pytest.mark.parametrize("scale", [1.0, 1e-7])
def test_nearly_dependent_column_is_kept_when_its_residual_is_resolved(scale):
    """A second column whose residual after the projection is 1e-3 of its length is a
    direction of its own: it is normalised, orthogonal to the first to 1e-12, and the step
    is the projector step on both (numpy).  One whose residual is 1e-6 of its length is
    dropped.  The decision is relative to the column's own length, so scaling the matrices
    by 1e-7 changes nothing."""
    rng = np.random.default_rng(43)
    n, m = 10, 8
    x1 = (rng.standard_normal((n, m)) * scale).astype(np.float32)
    x0 = (x1.astype(np.float64) + rng.standard_normal((n, m)) * scale).astype(np.float32)
    D = x0.astype(np.float64) - x1.astype(np.float64)
    q0 = rng.standard_normal(m)
    g = rng.standard_normal(m)

    def ratio_for(delta):
        qh = _unit_columns(np.stack([q0, q0 + delta * g], axis=1))
        P = D @ qh
        p0 = P[:, 0] / np.linalg.norm(P[:, 0])
        resid = P[:, 1] - (p0 @ P[:, 1]) * p0
        return np.linalg.norm(resid) / np.linalg.norm(P[:, 1])

    for target, expect_live in ((1e-3, True), (1e-6, False)):
        delta = target / ratio_for(1.0) if ratio_for(1.0) > 0 else target
        for _ in range(3):                                   # the ratio is linear in delta to first order
            delta *= target / ratio_for(delta)
        assert abs(ratio_for(delta) / target - 1.0) < 1e-3
        Q = np.stack([q0, q0 + delta * g], axis=1)
        o = _two_workers(n, m, rank=2)
        o.set_params(0, 0, x0)
        o.set_params(1, 0, x1)
        o.set_q(0, 1, 0, Q)
        o.round()
        P = o.get_phat(0, 1, 0)
        assert abs(o.min_residual_ratio() / target ** 2 - 1.0) < 1e-2       # the diagnostic is that ratio, squared
        w64 = float(np.float32(0.3))
        Ph = np.linalg.qr(D @ _unit_columns(Q))[0][:, :2 if expect_live else 1]
        proj = Ph @ Ph.T
        tol = 1e-9 * scale                                   # the second direction is resolved to 1e-16 / 1e-3
        assert np.allclose(o.get_params(0, 0), x0 - w64 * proj @ D, rtol=0, atol=tol)
        assert np.allclose(o.get_params(1, 0), x1 + w64 * proj @ D, rtol=0, atol=tol)
        if expect_live:
            assert abs(np.linalg.norm(P[:, 1]) - 1.0) < 1e-12 and abs(P[:, 0] @ P[:, 1]) < 1e-12
            assert not np.array_equal(o.get_q(0, 1, 0)[:, 1], Q[:, 1])
        else:
            assert np.array_equal(P[:, 1], np.zeros(n))
            assert np.array_equal(o.get_q(0, 1, 0)[:, 1], Q[:, 1])
        o.close()


def _workload_oracle(w):
    from paper_2008_01425_b200 import workloads as wl

    o = po.Oracle(kind=w.kind, n_workers=w.n_workers, layer_shapes=w.layer_shapes, rank=w.rank,
                  power_steps=w.power_steps, seed=w.seed, torus_rows=w.torus_rows, torus_cols=w.torus_cols,
                  custom_edges=w.custom_edges, weight_rule=w.weight_rule, W=wl.mixing_matrix(w))
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            o.set_params(i, l, wl.initial_params(w, i, l))
    return o


def test_no_workload_comes_near_the_dependent_column_threshold():
    """On the synthetic stacks that run at rank > 1 (the VGG-shaped ring at rank 2, and the
    torus and ResNet-20 recipes pushed to rank 2 and 4) the smallest residual ratio ever met
    stays above 1e-8, a hundred times the threshold of 1e-10; exactly dependent columns sit
    below 1e-24 (previous test).  Nothing lies in between, so any threshold from 1e-24 to 1e-8
    takes the same decisions on these inputs and gives the same trajectories."""
    from paper_2008_01425_b200 import workloads as wl

    small_vgg = [(max(n // 8, 3), max(m // 8, 5)) for n, m in wl.VGG16_SHAPES]
    cases = [
        wl.shrink(wl.vgg16_ring16(2), small_vgg, 50),
        wl.shrink(wl.vgg16_ring16(2), [(n // 4, m // 4) for n, m in wl.VGG16_SHAPES[4:9]], 6),
        wl.shrink(wl.torus8x8(2), [(200, 136)], 40).replace(rank=2),
        wl.shrink(wl.torus8x8(1), [(64, 48)], 60).replace(rank=4, torus_rows=3, torus_cols=3, n_workers=9),
        wl.resnet20_ring8().replace(rank=2, rounds=30,
                                    layer_shapes=tuple(s for s in wl.RESNET20_SHAPES if min(s) >= 2)),
    ]
    for w in cases:
        assert all(min(n, m) >= w.rank for n, m in w.layer_shapes)
        o = _workload_oracle(w)
        o.round(w.rounds)
        smallest = o.min_residual_ratio()
        o.close()
        assert smallest > 1e-8, (w.name, smallest)


def test_fp32_storage_emulation_only_rounds_the_state():
    """The test aid that rounds X and the stored vectors to fp32 after every power step:
    after a step the state is exactly the fp32 rounding of the untouched run's state, and
    it holds nothing but fp32 values."""
    rng = np.random.default_rng(47)
    a = _two_workers(9, 6, rank=2)
    b = _two_workers(9, 6, rank=2)
    b.set_fp32_storage()
    for o in (a, b):
        _fill(o, np.random.default_rng(47))
    a.round()
    b.round()
    for i in range(2):
        assert np.array_equal(b.get_params(i, 0), a.get_params(i, 0).astype(np.float32).astype(np.float64))
    assert np.array_equal(b.get_q(0, 1, 0), a.get_q(0, 1, 0).astype(np.float32).astype(np.float64))
    b.round(3)
    assert np.array_equal(b.get_params(0, 0), b.get_params(0, 0).astype(np.float32).astype(np.float64))
    a.close()
    b.close()
    del rng


# --------------------------------------------------------------------------
# Algorithm 2 read literally: one mat-vec and one update per iteration
# --------------------------------------------------------------------------
def _pair(n, m, w_edge, iterations, seed=3):
    W = np.array([[1 - w_edge, w_edge], [w_edge, 1 - w_edge]], dtype=np.float32)
    o = po.Oracle(kind=po.CUSTOM, n_workers=2, custom_edges=[(0, 1)], layer_shapes=[(n, m)], rank=1,
                  power_steps=iterations, seed=seed, weight_rule=po.W_EXPLICIT, W=W)
    o.set_half_step()
    return o


def test_half_step_mode_needs_rank_one_and_a_static_graph():
    o = po.Oracle(kind=po.RING, n_workers=4, layer_shapes=[(5, 4)], rank=2, power_steps=1, seed=1,
                  weight_rule=po.W_UNIFORM)
    with pytest.raises(ValueError):
        o.set_half_step()
    o = po.Oracle(kind=po.MATCHING, n_workers=4, layer_shapes=[(5, 4)], rank=1, power_steps=1, seed=1)
    with pytest.raises(ValueError):
        o.set_half_step()


@pytest.mark.parametrize("case", [CASES[0], CASES[1], CASES[5],
                                  dict(kind=po.TORUS, n_workers=12, torus_rows=3, torus_cols=4,
                                       layer_shapes=[(10, 8)], rank=1, power_steps=3,
                                       weight_rule=po.W_METROPOLIS)])
def test_half_step_average_conserved_and_distance_never_grows(case):
    """Lemma 1 holds for every iteration's update; a projection along a unit vector on
    either side is still a projector, so the consensus distance cannot grow."""
    rng = np.random.default_rng(4)
    o = po.Oracle(seed=19, **case)
    o.set_half_step()
    _fill(o, rng)
    avg0 = [o.average(l) for l in range(len(o.layer_shapes))]
    d_prev = o.consensus_distance()
    for _ in range(10):
        o.round()
        for l in range(len(o.layer_shapes)):
            assert np.abs(o.average(l) - avg0[l]).max() <= 1e-13 * max(np.abs(avg0[l]).max(), 1.0)
        d = o.consensus_distance()
        assert d <= d_prev * (1 + 1e-12)
        d_prev = d
    o.close()


def test_half_step_vector_alternates_between_the_two_spaces():
    """After an odd iteration the pair's vector lives in R^rows, after an even one in
    R^cols (Algorithm 2's comment), so an iteration moves (rows+cols)/2 floats on
    average: the count behind the printed per-tensor compression ratios."""
    n, m = 64, 576
    o = _pair(n, m, 0.25, 1)
    _fill(o, np.random.default_rng(0))
    lengths = []
    for _ in range(6):
        o.round()
        lengths.append(len(o.get_vector(0, 1, 0)))
    assert lengths == [n, m, n, m, n, m]
    assert round(n * m / np.mean(lengths)) == 115            # the ResNet-20 table prints 115/r
    o.close()


def test_half_step_removes_a_rank_one_difference_in_two_iterations():
    """D = sigma u v^T: the odd iteration leaves a difference that is still u times a
    row vector and makes the stored vector parallel to u; the even iteration's
    approximation vh vh^T D is then exact, so with W = 1/2 both ends meet at their
    average after two iterations."""
    rng = np.random.default_rng(6)
    n, m = 9, 7
    base = np.round(rng.standard_normal((n, m)) * 64) / 64
    u = np.round(rng.standard_normal((n, 1)) * 8) / 8
    v = np.round(rng.standard_normal((1, m)) * 8) / 8
    x0, x1 = (base + u @ v).astype(np.float32), base.astype(np.float32)
    o = _pair(n, m, 0.5, 2)
    o.set_params(0, 0, x0)
    o.set_params(1, 0, x1)
    o.round()
    mean = (x0.astype(np.float64) + x1.astype(np.float64)) / 2
    assert np.allclose(o.get_params(0, 0), mean, rtol=0, atol=1e-13)
    assert np.allclose(o.get_params(1, 0), mean, rtol=0, atol=1e-13)
    # after ONE iteration they have not met yet (unless v happens to be parallel to the seed vector)
    o2 = _pair(n, m, 0.5, 1)
    o2.set_params(0, 0, x0)
    o2.set_params(1, 0, x1)
    o2.round()
    assert not np.allclose(o2.get_params(0, 0), mean, rtol=0, atol=1e-6)
    o.close()
    o2.close()


def test_half_step_on_a_frozen_difference_is_power_iteration():
    """Eq. 3 with D fixed (edge weight 0): the stored vector converges to sigma_1 u_1 after odd
    iterations and sigma_1 v_1 after even ones (numpy.linalg.svd)."""
    rng = np.random.default_rng(12)
    n, m = 8, 6
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    V, _ = np.linalg.qr(rng.standard_normal((m, m)))
    sv = np.array([4.0, 2.0, 1.0, 0.5, 0.2, 0.1])
    x1 = rng.standard_normal((n, m)).astype(np.float32)
    x0 = (x1 + (U[:, :m] * sv) @ V.T).astype(np.float32)
    D = x0.astype(np.float64) - x1.astype(np.float64)
    Us, ss, Vts = np.linalg.svd(D)
    o = _pair(n, m, 0.0, 1)
    o.set_params(0, 0, x0)
    o.set_params(1, 0, x1)
    for it in range(1, 61):
        o.round()
    vec = o.get_vector(0, 1, 0)                 # 60 iterations: even, so in R^cols
    assert len(vec) == m
    assert abs(np.linalg.norm(vec) - ss[0]) < 1e-8 * ss[0]
    assert abs(abs(vec @ Vts[0]) - ss[0]) < 1e-8 * ss[0]
    o.round()
    vec = o.get_vector(0, 1, 0)                 # odd: in R^rows
    assert len(vec) == n
    assert abs(abs(vec @ Us[:, 0]) - ss[0]) < 1e-8 * ss[0]
    assert np.array_equal(o.get_params(0, 0), x0.astype(np.float64))
    o.close()


def test_half_step_first_iteration_on_single_column_layers_is_plain_gossip():
    """For an n x 1 tensor the first (odd) iteration projects on a 1-vector, which
    reproduces every difference exactly: one uncompressed gossip step X <- W X
    (Eq. 1's averaging term), on a ring with all edges acting at once."""
    rng = np.random.default_rng(14)
    N, n = 6, 7
    W = _ring_W(N, 0.3)
    o = po.Oracle(kind=po.RING, n_workers=N, layer_shapes=[(n, 1)], rank=1, power_steps=1,
                  seed=23, weight_rule=po.W_EXPLICIT, W=W)
    o.set_half_step()
    xs = _fill(o, rng)
    X = np.stack([xs[i][0] for i in range(N)])
    o.round()
    expect = np.einsum("ij,jnm->inm", W.astype(np.float64), X)
    got = np.stack([o.get_params(i, 0) for i in range(N)])
    assert np.allclose(got, expect, rtol=0, atol=1e-12)
    o.close()


@pytest.mark.parametrize("shape", [(7, 1), (1, 7)])
@pytest.mark.parametrize("iterations", [2, 3, 4])
def test_half_step_isolated_pair_single_column_or_row(shape, iterations):
    """Two workers, an n x 1 (or 1 x m) tensor: the difference keeps its direction, so
    every iteration whose unit vector lives in the 1-dimensional space is exact and
    the others project a vector on itself: the difference shrinks by (1 - 2W) per
    exact iteration.  n x 1: all iterations exact.  1 x m: the first (odd) one
    projects the row on the seed direction, all later ones are exact."""
    rng = np.random.default_rng(15)
    wgt = 0.3
    o = _pair(shape[0], shape[1], wgt, iterations)
    xs = _fill(o, rng)
    D0 = xs[0][0] - xs[1][0]
    o.round()
    D = o.get_params(0, 0) - o.get_params(1, 0)
    w64 = float(np.float32(wgt))
    if shape[1] == 1:
        assert np.allclose(D, (1 - 2 * w64) ** iterations * D0, rtol=0, atol=1e-13)
    else:
        q = po.init_q(3, 0, 1, 0, 0, shape[1]).astype(np.float64)
        q /= np.linalg.norm(q)
        D1 = D0 - 2 * w64 * (D0 @ q)[:, None] * q[None, :]          # after the first iteration
        assert np.allclose(D, (1 - 2 * w64) ** (iterations - 1) * D1, rtol=0, atol=1e-13)
    o.close()


def test_half_step_identical_workers_stay_put():
    x = np.random.default_rng(2).standard_normal((6, 5)).astype(np.float32)
    o = po.Oracle(kind=po.RING, n_workers=4, layer_shapes=[(6, 5)], rank=1, power_steps=3, seed=4,
                  weight_rule=po.W_UNIFORM)
    o.set_half_step()
    for i in range(4):
        o.set_params(i, 0, x)
    o.round(2)
    for i in range(4):
        assert np.array_equal(o.get_params(i, 0), x.astype(np.float64))
    o.close()


# --------------------------------------------------------------------------
# random-projection compressors (Section 5.1): R_k(X) = (X U) U^T,  L_k(X) = V (V^T X)
# --------------------------------------------------------------------------
def test_random_directions_are_orthonormal_keyed_and_uniform():
    """u ~ uniform on the sphere means E[u u^T] = I/len, and for k orthonormal columns
    E[U U^T] = (k/len) I: the delta of assumption A5."""
    U = po.random_directions(9, 0, 0, 1, 0, 40, 4)
    assert np.allclose(U.T @ U, np.eye(4), atol=1e-12)
    assert np.array_equal(U, po.random_directions(9, 0, 0, 1, 0, 40, 4))
    for other in (po.random_directions(9, 1, 0, 1, 0, 40, 4), po.random_directions(10, 0, 0, 1, 0, 40, 4),
                  po.random_directions(9, 0, 0, 2, 0, 40, 4), po.random_directions(9, 0, 0, 1, 1, 40, 4)):
        assert np.abs(other - U).max() > 0.05
    for k in (1, 2):
        acc = np.zeros((6, 6))
        T = 6000
        for t in range(T):
            V = po.random_directions(3, t, 0, 1, 0, 6, k)
            acc += V @ V.T
        assert np.abs(acc / T - (k / 6.0) * np.eye(6)).max() < 0.02
    # more columns than dimensions: the surplus columns are dropped
    V = po.random_directions(3, 0, 0, 1, 0, 2, 4)
    assert np.allclose(V[:, :2].T @ V[:, :2], np.eye(2), atol=1e-12) and np.all(V[:, 2:] == 0)


@pytest.mark.parametrize("mode", [po.RANDOM_RIGHT, po.RANDOM_LEFT])
@pytest.mark.parametrize("case", [CASES[1], CASES[2], CASES[3]])
def test_random_projection_average_conserved_and_distance_never_grows(mode, case):
    rng = np.random.default_rng(8)
    o = po.Oracle(seed=29, **case)
    o.set_random_projection(mode)
    _fill(o, rng)
    avg0 = [o.average(l) for l in range(len(o.layer_shapes))]
    d_prev = o.consensus_distance()
    for _ in range(8):
        o.round()
        for l in range(len(o.layer_shapes)):
            assert np.abs(o.average(l) - avg0[l]).max() <= 1e-13 * max(np.abs(avg0[l]).max(), 1.0)
        d = o.consensus_distance()
        assert d <= d_prev * (1 + 1e-12)
        d_prev = d
    o.close()


@pytest.mark.parametrize("mode,shape,rank", [(po.RANDOM_RIGHT, (7, 3), 3), (po.RANDOM_RIGHT, (5, 1), 1),
                                             (po.RANDOM_LEFT, (3, 7), 3), (po.RANDOM_LEFT, (2, 9), 4)])
def test_random_projection_with_a_full_basis_is_plain_gossip(mode, shape, rank):
    """k = cols (right) or k = rows (left): U U^T = I, so the step is X <- W X (Eq. 1)."""
    rng = np.random.default_rng(16)
    N = 6
    W = _ring_W(N, 0.3)
    o = po.Oracle(kind=po.RING, n_workers=N, layer_shapes=[shape], rank=rank, power_steps=1, seed=33,
                  weight_rule=po.W_EXPLICIT, W=W)
    o.set_random_projection(mode)
    xs = _fill(o, rng)
    X = np.stack([xs[i][0] for i in range(N)])
    o.round()
    expect = np.einsum("ij,jnm->inm", W.astype(np.float64), X)
    got = np.stack([o.get_params(i, 0) for i in range(N)])
    assert np.allclose(got, expect, rtol=0, atol=1e-12)
    o.close()


@pytest.mark.parametrize("mode", [po.RANDOM_RIGHT, po.RANDOM_LEFT])
def test_random_projection_one_step_is_the_projector_update(mode):
    """Eq. (compressed consensus): X_i += sum_j W_ij (C(X_j) - C(X_i)) with the step's own directions."""
    rng = np.random.default_rng(21)
    N, n, m, k = 5, 7, 9, 2
    W = _ring_W(N, 0.25)
    o = po.Oracle(kind=po.RING, n_workers=N, layer_shapes=[(n, m)], rank=k, power_steps=1, seed=41,
                  weight_rule=po.W_EXPLICIT, W=W)
    o.set_random_projection(mode)
    xs = _fill(o, rng)
    X = [xs[i][0] for i in range(N)]
    edges, w = o.round_schedule()
    new = [x.copy() for x in X]
    for (i, j), wij in zip(edges, w):
        if mode == po.RANDOM_RIGHT:
            U = po.random_directions(41, 0, i, j, 0, m, k)
            C = lambda A: (A @ U) @ U.T
        else:
            V = po.random_directions(41, 0, i, j, 0, n, k)
            C = lambda A: V @ (V.T @ A)
        new[i] += wij * (C(X[j]) - C(X[i]))
        new[j] += wij * (C(X[i]) - C(X[j]))
    o.round()
    for i in range(N):
        assert np.allclose(o.get_params(i, 0), new[i], rtol=0, atol=1e-12)
    o.close()


def test_random_projection_directions_are_fresh_every_step():
    """An isolated pair with W = 1/2 loses the component of D along u entirely at every
    step; with fresh directions E||D||^2 shrinks by (1 - 1/cols) per step, so D vanishes."""
    o = _pair(5, 6, 0.5, 1)
    o.set_half_step(False)
    o.set_random_projection(po.RANDOM_RIGHT)
    xs = _fill(o, np.random.default_rng(3))
    d0 = np.linalg.norm(xs[0][0] - xs[1][0])
    o.round(250)
    assert np.linalg.norm(o.get_params(0, 0) - o.get_params(1, 0)) < 1e-6 * d0
    o.close()


def test_theorem_1_contraction_in_expectation():
    """Theorem 1: E sum_i ||X_i - mean||^2 shrinks by at least (1 - rho delta) per step,
    rho = 1 - lambda_2(W)^2, delta = k/cols for R_k.  Averaged over 400 direction seeds."""
    rng = np.random.default_rng(31)
    N, n, m, k = 6, 4, 6, 1
    W = _ring_W(N, 0.3)
    lam = np.sort(np.abs(np.linalg.eigvalsh(W.astype(np.float64))))[::-1]
    rho, delta = 1.0 - lam[1] ** 2, k / m
    X = [(rng.standard_normal((n, m))).astype(np.float32) for _ in range(N)]
    ratios = []
    for seed in range(400):
        o = po.Oracle(kind=po.RING, n_workers=N, layer_shapes=[(n, m)], rank=k, power_steps=1, seed=seed,
                      weight_rule=po.W_EXPLICIT, W=W)
        o.set_random_projection(po.RANDOM_RIGHT)
        for i in range(N):
            o.set_params(i, 0, X[i])
        d0 = o.consensus_distance()
        o.round()
        ratios.append(o.consensus_distance() / d0)
        o.close()
    ratios = np.array(ratios)
    sem = ratios.std() / np.sqrt(len(ratios))
    assert ratios.mean() <= (1.0 - rho * delta) + 3 * sem
    assert ratios.mean() < 1.0 - 0.5 * rho * delta        # and it does contract
