"""Parity of the CUDA path against the fp64 CPU checker, through the C ABI.

Tolerance: max over (worker, layer) of ||X_gpu - X_ref||_F / ||X_ref||_F <= 1e-4,
and the worker average on the GPU moves by at most 1e-5 relative (Lemma 1 is
exact in exact arithmetic; fp32 rounding of +u and -u differs).  Schedules are
compared bit for bit.

The warm-started, deflating power iteration is a chaotic map on noise-like
differences: two fp64 runs of the checker whose initial vectors differ by 1e-12
are 4e-2 apart after 100 rounds of the ResNet-20 workload (tests/test_chaos.py
measures this on the CPU).  fp32 storage of X perturbs every step by 6e-8, so a
free-running fp32 run can follow the fp64 trajectory to 1e-4 only over a limited
horizon.  Hence two kinds of test:
  free-running   both sides start from the same bits and run without contact;
                 1e-4 is asserted up to the horizon stated per workload, and at
                 the full round count the invariants (average conserved,
                 consensus distance close to the checker's) are asserted;
  re-based       every few power steps the checker's own state is rounded to
                 fp32 and loaded into both sides, and 1e-4 is asserted over the
                 whole stated number of rounds.  This checks every round of the
                 computation along the checker's trajectory.
"""
import numpy as np
import pytest

from paper_2008_01425_b200 import workloads as wl
from tests import common

pytestmark = pytest.mark.gpu

REL_TOL = 1e-4
CHANGE_TOL = 1e-3            # the same error against ||X_ref - X_start||_F, what the rounds changed
                             # (matrices whose error is below common.FP32_FLOOR of ||X|| are exempt)
CHANGE_TOL_REBASED = 1e-2    # re-based segments: late ones change X by little, and on matrices of a few
                             # dozen entries the direction found is ill-conditioned (1.7e-3 met on an 8 x 5 layer)
AVG_TOL = 1e-5
SEGMENT_POWER_STEPS = 8      # re-base at least this often (in power steps)


def _check_schedules(oracle, net, rounds):
    for t in sorted({0, 1, max(rounds - 1, 0)}):
        e_ref, w_ref = oracle.round_schedule(t)
        e_gpu, w_gpu = net.pg_get_schedule(t)
        assert np.array_equal(e_gpu, e_ref)
        assert np.array_equal(w_gpu, w_ref.astype(np.float32))


def _check_average(w, net, avg0):
    for l in range(len(w.layer_shapes)):
        drift = np.linalg.norm(common.gpu_average(w, net, l) - avg0[l]) / max(np.linalg.norm(avg0[l]), 1e-300)
        assert drift <= AVG_TOL, "layer %d: average drift %.3e" % (l, drift)


ENVELOPE = 3.0               # the GPU may drift this many times further than fp32 storage alone (1.5 met)


def _gap(w, a, b):
    """max over (worker, layer) of ||X_a - X_b||_F / ||X_b||_F between two CPU checkers."""
    worst = 0.0
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            ref = b.get_params(i, l)
            worst = max(worst, float(np.linalg.norm(a.get_params(i, l) - ref) / max(np.linalg.norm(ref), 1e-300)))
    return worst


def _run(w, rounds=None, check_every=None, horizon=None, rebased=False, distance_tol=0.05, envelope=False):
    """Run `rounds` rounds on both sides.

    free-running (rebased=False): assert 1e-4 (on ||X||) and 1e-3 (on what the rounds
    changed since the seeded start) at every check up to round `horizon` (default: all
    rounds); past the horizon only the invariants.
    rebased=True: re-base every SEGMENT_POWER_STEPS power steps, assert 1e-4 at the end of
    every segment, and 1e-2 on what the segment changed since the state it started from.
    envelope=True (free-running): a second fp64 checker runs beside the first with its state
    rounded to fp32 after every power step, the least any fp32-storage implementation of
    Algorithm 2 perturbs the iteration.  At the full round count the GPU's distance from the
    untouched fp64 run must be within 1e-4, or within ENVELOPE times that checker's distance.
    One line per run with the largest of either figure goes to the end of the pytest log.
    """
    from paper_2008_01425_b200 import binding as pg

    rounds = w.rounds if rounds is None else rounds
    horizon = rounds if horizon is None else horizon
    oracle = common.oracle_for(w)
    net = common.network_for(w)
    common.load_both(w, oracle, net)
    shadow = None
    if envelope:
        shadow = common.oracle_for(w)
        shadow.set_fp32_storage()
        common.load_both(w, shadow, None)
    _check_schedules(oracle, net, rounds)
    avg0 = [common.initial_average(w, l) for l in range(len(w.layer_shapes))]
    if rebased:
        check_every = max(1, SEGMENT_POWER_STEPS // w.power_steps)
    pairs = set()
    done, err = 0, 0.0
    worst_x, worst_change, start = 0.0, 0.0, None
    while done < rounds:
        step = rounds - done if not check_every else min(check_every, rounds - done)
        for t in range(done, done + step):
            pairs.update((int(a), int(b)) for a, b in oracle.round_schedule(t)[0])
            net.pg_round()
        oracle.round(step)
        if shadow is not None:
            shadow.round(step)
        done += step
        if rebased or done <= horizon:
            (err, where), (err_c, where_c) = common.relative_errors(w, oracle, net, start)
            worst_x, worst_change = max(worst_x, err), max(worst_change, err_c)
            assert err <= REL_TOL, "round %d: relative error %.3e at (worker, layer) %r" % (done, err, where)
            assert err_c <= (CHANGE_TOL_REBASED if rebased else CHANGE_TOL), (
                "round %d: error %.3e of what the rounds changed at (worker, layer) %r" % (done, err_c, where_c))
        if rebased and done < rounds:
            start = common.rebase(w, oracle, net, pairs)
    assert net.pg_device_status() == pg.PG_OK
    assert net.pg_get_round() == rounds
    if not rebased:
        _check_average(w, net, avg0)
        d_ref, d_gpu = oracle.consensus_distance(), common.gpu_consensus_distance(w, net)
        assert abs(d_gpu - d_ref) <= distance_tol * d_ref, (d_gpu, d_ref)
    note = ""
    if shadow is not None:
        gap_gpu, where = common.max_relative_error(w, oracle, net)
        gap_shadow = _gap(w, shadow, oracle)
        assert gap_gpu <= max(REL_TOL, ENVELOPE * gap_shadow), (gap_gpu, gap_shadow, where)
        note += "; at round %d: GPU %.2e from the fp64 run, fp64 arithmetic with fp32 storage %.2e" % (
            rounds, gap_gpu, gap_shadow)
        shadow.close()
    if w.rank > 1 and all(min(n, m) >= w.rank for n, m in w.layer_shapes):
        # no Gram-Schmidt residual came near the dependent-column threshold (1e-10): both sides
        # took the same decisions whatever the threshold's exact value
        smallest = oracle.min_residual_ratio()
        assert smallest > 1e-8, smallest
        note += ", smallest residual ratio %.1e" % smallest
    common.PARITY_LINES.append(
        "%-34s rank %d %s %3d rounds: max error %.2e of ||X||, %.2e of the change%s"
        % (w.name, w.rank, "re-based" if rebased else "free-run", rounds, worst_x, worst_change,
           "" if rebased or horizon >= rounds else " (asserted to round %d, invariants after)" % horizon) + note)
    net.close()
    oracle.close()
    return err


def test_config1_tiny_ring():
    _run(wl.tiny_ring(), check_every=5)


def test_config2_resnet20_ring8_free_running():
    """All 100 rounds; the fp64 trajectory can be followed to 1e-4 for 20 rounds."""
    _run(wl.resnet20_ring8(), check_every=10, horizon=20, envelope=True)


def test_config2_resnet20_ring8_rebased():
    _run(wl.resnet20_ring8(), rebased=True)


@pytest.mark.parametrize("power_steps", [1, 2, 4])
def test_config3_torus_small_rebased(power_steps):
    """The torus workload on 200 x 136 matrices (several tiles, ragged tails), all 200 rounds."""
    _run(wl.shrink(wl.torus8x8(power_steps), [(200, 136)], 200), rebased=True)


@pytest.mark.parametrize("power_steps", [1, 2, 4])
def test_config3_torus_small_free_running(power_steps):
    w = wl.shrink(wl.torus8x8(power_steps), [(200, 136)], 200)
    _run(w, check_every=max(1, 20 // power_steps), horizon=20 // power_steps, envelope=True)


def test_config3_torus_full_size_free_running():
    w = wl.torus8x8(1)
    _run(w, check_every=20, horizon=20, envelope=True)


@pytest.mark.parametrize("power_steps", [1, 2, 4])
def test_config3_torus_full_size_rebased(power_steps):
    w = wl.torus8x8(power_steps)
    _run(w, rebased=True)


@pytest.mark.parametrize("rank", [1, 2])
def test_config4_vgg16_ring16_full_size(rank):
    w = wl.vgg16_ring16(rank)
    _run(w, rebased=True)


@pytest.mark.parametrize("rank", [1, 2])
def test_config4_vgg16_ring16_full_size_free_running(rank):
    """All 50 rounds without contact: 1e-4 asserted over the first rounds, then the invariants
    and the fp32-storage envelope."""
    _run(wl.vgg16_ring16(rank), check_every=5, horizon=5, envelope=True)


@pytest.mark.parametrize("rank", [1, 2])
def test_config4_vgg16_small_rebased(rank):
    """VGG-shaped stack with every layer shrunk 8x per side: all 50 rounds."""
    shapes = [(max(n // 8, 3), max(m // 8, 5)) for n, m in wl.VGG16_SHAPES]
    _run(wl.shrink(wl.vgg16_ring16(rank), shapes, 50), rebased=True)


@pytest.mark.parametrize("rank", [1, 2])
def test_config4_vgg16_small_free_running(rank):
    shapes = [(max(n // 8, 3), max(m // 8, 5)) for n, m in wl.VGG16_SHAPES]
    _run(wl.shrink(wl.vgg16_ring16(rank), shapes, 50), check_every=5, horizon=5, envelope=True)


def test_config5_lstm_matching_small():
    """The time-varying matching workload with a 1/10-scale stack, all 20 rounds, free-running."""
    shapes = [(2800, 65)] + [(260, 65)] * 6 + [(65, 2800)]
    _run(wl.shrink(wl.lstm_matching32(), shapes, 20), check_every=5)


def test_config5_lstm_matching_small_rebased():
    shapes = [(2800, 65)] + [(260, 65)] * 6 + [(65, 2800)]
    _run(wl.shrink(wl.lstm_matching32(), shapes, 20), rebased=True)


def test_config5_lstm_matching_full_size():
    """Full 5.96 GB stack, free-running; the checker needs about 12 GB of host memory."""
    w = wl.lstm_matching32()
    _run(w, check_every=10)


# ---- edge cases -------------------------------------------------------------
EDGE_SHAPES = [
    [(1, 1)], [(1, 9)], [(9, 1)], [(5, 3)], [(3, 5)], [(67, 131)], [(300, 7)], [(7, 2500)],
    [(64, 27), (10, 64), (33, 130)],
]


@pytest.mark.parametrize("shapes", EDGE_SHAPES)
@pytest.mark.parametrize("rank", [1, 2, 4])
def test_ragged_and_degenerate_shapes(shapes, rank):
    """Columns not a multiple of 4, single rows / columns, rank above min(rows, cols)."""
    w = wl.Workload("edge", 9, 4, wl.RING, 0, 0, wl.W_EXPLICIT, 0.3, tuple(shapes), rank, 2, 6, 77, "normal1")
    _run(w, rebased=True)
    _run(w, rounds=2)


@pytest.mark.parametrize("kind", ["torus_deg4_rank2", "torus_2x4", "custom_star", "matching2"])
def test_graph_variants(kind):
    if kind == "torus_deg4_rank2":
        w = wl.Workload("t", 9, 9, wl.TORUS, 3, 3, wl.W_METROPOLIS, None, ((40, 52),), 2, 1, 10, 5, "normal1")
    elif kind == "torus_2x4":
        w = wl.Workload("t", 9, 8, wl.TORUS, 2, 4, wl.W_UNIFORM, None, ((40, 52),), 1, 2, 10, 5, "normal1")
    elif kind == "custom_star":
        w = wl.Workload("t", 9, 5, wl.CUSTOM, 0, 0, wl.W_METROPOLIS, None, ((40, 52), (8, 8)), 1, 1, 10, 5,
                        "normal1", custom_edges=((0, 1), (0, 2), (0, 3), (3, 4)))
    else:
        w = wl.Workload("t", 9, 2, wl.MATCHING, 0, 0, wl.W_METROPOLIS, None, ((40, 52),), 1, 1, 4, 5, "normal1")
    _run(w, rebased=True)
    _run(w, rounds=4)


@pytest.mark.parametrize("rank", [1, 2])
def test_whole_tiles_on_workers_with_fewer_edges_than_slots(rank):
    """A star with a tail: degrees 3, 1, 1, 2, 1 under kernels built for four (rank 1) or eight (rank 2)
    vectors, on matrices whose tiles are whole row batches and column steps, so the sweeps take their
    forms without conditions and work on the vectors a worker lacks as zeros."""
    w = wl.Workload("t", 9, 5, wl.CUSTOM, 0, 0, wl.W_METROPOLIS, None, ((64, 256), (32, 128), (128, 384)), rank, 2, 6, 5,
                    "normal1", custom_edges=((0, 1), (0, 2), (0, 3), (3, 4)))
    _run(w, rebased=True)
    _run(w, rounds=3)


def test_identical_workers_stay_bit_identical():
    """Consensus is a fixed point (Section 4.1): nothing moves, nothing is NaN."""
    w = wl.Workload("same", 9, 6, wl.RING, 0, 0, wl.W_UNIFORM, None, ((33, 70),), 2, 2, 3, 5, "normal1")
    net = common.network_for(w)
    x = wl.initial_params(w, 0, 0)
    for i in range(w.n_workers):
        net.pg_write_params(i, 0, x)
    q0 = net.pg_read_q(0, 1, 0)
    for _ in range(3):
        net.pg_round()
    for i in range(w.n_workers):
        assert np.array_equal(net.pg_read_params(i, 0), x)
    assert np.array_equal(net.pg_read_q(0, 1, 0), q0)
    net.close()


def test_non_finite_parameters_raise_the_status_word():
    from paper_2008_01425_b200 import binding as pg

    w = wl.Workload("nan", 9, 4, wl.RING, 0, 0, wl.W_UNIFORM, None, ((16, 16),), 1, 1, 1, 5, "normal1")
    net = common.network_for(w)
    common.load_both(w, None, net)
    x = wl.initial_params(w, 1, 0)
    x[3, 3] = np.inf
    net.pg_write_params(1, 0, x)
    net.pg_round()
    assert net.pg_device_status() == pg.PG_ERR_NUMERIC
    net.close()


def test_runs_are_bit_reproducible_and_checkpoint_resumes():
    """Fixed-order reductions: two runs agree bit for bit; {X, Q, round} is a full checkpoint."""
    w = wl.shrink(wl.lstm_matching32(), [(130, 70), (70, 130)], 8).replace(n_workers=8)
    def fresh():
        net = common.network_for(w)
        common.load_both(w, None, net)
        return net
    a, b = fresh(), fresh()
    for _ in range(4):
        a.pg_round()
        b.pg_round()
    snap_x = a.read_all()
    snap_q = {(i, j): [a.pg_read_q(i, j, l) for l in range(2)] for i in range(8) for j in range(i + 1, 8)}
    for _ in range(4):
        a.pg_round()
        b.pg_round()
    xa, xb = a.read_all(), b.read_all()
    c = common.network_for(w)
    c.write_all(snap_x)
    for (i, j), qs in snap_q.items():
        for l, q in enumerate(qs):
            c.pg_write_q(i, j, l, q)
    c.pg_set_round(4)
    for _ in range(4):
        c.pg_round()
    xc = c.read_all()
    for i in range(8):
        for l in range(2):
            assert np.array_equal(xa[i][l], xb[i][l])
            assert np.array_equal(xa[i][l], xc[i][l])
    for n in (a, b, c):
        n.close()


@pytest.mark.parametrize("w", [wl.tiny_ring(), wl.shrink(wl.torus8x8(2), [(200, 136)], 6),
                               wl.shrink(wl.lstm_matching32(), [(130, 70), (70, 1300)], 6).replace(n_workers=8)],
                         ids=lambda w: w.name)
def test_dependent_launches_do_not_change_a_bit(w, monkeypatch):
    """Kernels scheduled during the previous kernel's tail wait for it on the device before they
    touch memory: the run ends on the bits of a run with plain launches."""
    def run():
        net = common.network_for(w)
        common.load_both(w, None, net)
        for _ in range(w.rounds):
            net.pg_round()
        x = net.read_all()
        assert net.pg_device_status() == 0
        net.close()
        return x
    xa = run()
    monkeypatch.setenv("PG_DEPENDENT_LAUNCH", "0")
    xb = run()
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            assert np.array_equal(xa[i][l], xb[i][l])


def test_async_read_back_beside_the_next_upload():
    """Upload, round, read back, several times over: the read-back of one result on one
    stream beside the upload of the next input on another (each matrix gated on its own
    event) ends on the same bits as the blocking calls on one stream."""
    import torch

    w = wl.shrink(wl.lstm_matching32(), [(130, 70), (70, 1300), (300, 652)], 4).replace(n_workers=8)
    L = len(w.layer_shapes)
    steps = 3
    rng = np.random.default_rng(77)
    inputs = [[[torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).pin_memory()
                for shape in w.layer_shapes] for _ in range(w.n_workers)] for _ in range(steps)]

    ref = common.network_for(w)
    expected = []
    for s in range(steps):
        for i in range(w.n_workers):
            for l in range(L):
                ref.pg_write_params(i, l, inputs[s][i][l])
        ref.pg_round()
        expected.append([[ref.pg_read_params(i, l) for l in range(L)] for i in range(w.n_workers)])
    ref.close()

    net = common.network_for(w)
    main = torch.cuda.current_stream()
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    out = [[[torch.empty(shape, dtype=torch.float32).pin_memory() for shape in w.layer_shapes]
            for _ in range(w.n_workers)] for _ in range(steps)]
    read_done = [[torch.cuda.Event() for _ in range(L)] for _ in range(w.n_workers)]
    for s in range(steps):
        for i in range(w.n_workers):
            for l in range(L):
                if s > 0:
                    up.wait_event(read_done[i][l])
                net.pg_write_params(i, l, inputs[s][i][l], up)
        main.wait_stream(up)
        net.pg_round(main)
        down.wait_stream(main)
        for i in range(w.n_workers):
            for l in range(L):
                net.pg_read_params_async(i, l, out[s][i][l], down)
                read_done[i][l].record(down)
    main.wait_stream(down)
    torch.cuda.synchronize()
    assert net.pg_device_status(main) == 0
    for s in range(steps):
        for i in range(w.n_workers):
            for l in range(L):
                assert np.array_equal(out[s][i][l].numpy(), expected[s][i][l]), (s, i, l)
    net.close()


def test_initial_vectors_on_device_are_the_seeded_ones():
    from oracle import pg_oracle as po

    w = wl.shrink(wl.lstm_matching32(), [(30, 70)], 1).replace(n_workers=6, rank=2)
    net = common.network_for(w)
    for (i, j) in [(0, 1), (2, 5), (4, 5)]:
        q = net.pg_read_q(i, j, 0)
        for k in range(2):
            assert np.array_equal(q[:, k], po.init_q(w.seed, i, j, 0, k, 70))
    net.close()


def test_communication_volume_of_a_round():
    """pg_comm_floats_round: both ends of every edge of the round send rank * rows floats per odd
    iteration of Algorithm 2 and rank * cols per even one, summed over the layers."""
    shapes = ((64, 32), (9, 5))
    rows, cols, dense = 64 + 9, 32 + 5, 64 * 32 + 9 * 5
    ring = wl.tiny_ring().replace(layer_shapes=shapes, rank=2, power_steps=3)
    net = common.network_for(ring)
    ends = 2 * 4                                            # ring of 4: four edges
    assert net.pg_comm_floats_round(0) == (ends * 2 * 3 * (rows + cols), ends * dense)
    assert net.pg_comm_floats_round(7) == net.pg_comm_floats_round(0)
    net.close()
    half = common.network_for(ring.replace(rank=1))
    half.pg_set_half_step()                                  # three iterations a round: k = 1, 2, 3, then 4, 5, 6
    assert half.pg_comm_floats_round(0)[0] == ends * (2 * rows + cols)
    assert half.pg_comm_floats_round(1)[0] == ends * (rows + 2 * cols)
    half.close()
    for mode, per_step in ((1, rows), (2, cols)):
        rp = common.network_for(ring)
        rp.pg_set_random_projection(mode)
        assert rp.pg_comm_floats_round(0)[0] == ends * 2 * 3 * per_step
        rp.close()
    match = common.network_for(wl.shrink(wl.lstm_matching32(), shapes, 1).replace(n_workers=6))
    assert match.pg_comm_floats_round(3) == (6 * (rows + cols), 6 * dense)       # three pairs, six ends
    match.close()


def test_set_round_on_the_stream_of_the_rounds():
    """A correction still pending when the round counter is set is applied on the stream the
    caller names; with the rounds on a non-blocking stream the result is that of the default one."""
    import torch

    w = wl.Workload("ring_set_round", 9, 5, wl.RING, 0, 0, wl.W_UNIFORM, None, ((70, 130), (24, 1500)), 1, 1, 4, 3,
                    "normal1")
    results = []
    for stream in (None, torch.cuda.Stream()):
        net = common.network_for(w)
        common.load_both(w, None, net)
        if stream is not None:
            stream.wait_stream(torch.cuda.current_stream())
        for _ in range(3):
            net.pg_round(stream)
        net.pg_set_round(1, stream)            # flushes the pending correction, then replays round 1's counter
        net.pg_round(stream)
        assert net.pg_get_round() == 2
        results.append(net.read_all(stream))
        net.close()
    for i in range(w.n_workers):
        for l in range(2):
            assert np.array_equal(results[0][i][l], results[1][i][l])


# ---- one cooperative launch for many rounds (small stacks) --------------------
PERSISTENT_CASES = [
    wl.tiny_ring(),
    wl.resnet20_ring8().replace(rounds=12),
    wl.shrink(wl.torus8x8(2), [(200, 136)], 6),
    wl.shrink(wl.vgg16_ring16(2), [(max(n // 8, 3), max(m // 8, 5)) for n, m in wl.VGG16_SHAPES], 5),
]


@pytest.mark.parametrize("w", PERSISTENT_CASES, ids=lambda w: w.name)
def test_pg_rounds_equals_repeated_pg_round_bit_for_bit(w, monkeypatch):
    """pg_rounds(n) runs the same arithmetic in the same order as n calls of pg_round.
    (Rank-1 rings would take the pair sweep, which pg_rounds enqueues round by round; switched
    off here so that the cooperative kernel is the one compared.)"""
    monkeypatch.setenv("PG_DISABLE_PAIR_SWEEP", "1")
    a, b = common.network_for(w), common.network_for(w)
    common.load_both(w, None, a)
    common.load_both(w, None, b)
    for _ in range(w.rounds):
        a.pg_round()
    b.pg_rounds(3)                 # starts with the stand-alone forward product
    b.pg_rounds(w.rounds - 3)      # continues from the cached one
    assert a.pg_get_round() == b.pg_get_round() == w.rounds
    assert a.pg_device_status() == 0 and b.pg_device_status() == 0
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            assert np.array_equal(a.pg_read_params(i, l), b.pg_read_params(i, l))
    e = a.pg_get_schedule(0)[0][0]
    assert np.array_equal(a.pg_read_q(int(e[0]), int(e[1]), 0), b.pg_read_q(int(e[0]), int(e[1]), 0))
    a.close()
    b.close()


REPLAY_CASES = [
    wl.tiny_ring(),                                   # pair sweep on a ring (two copies of X swap every step)
    wl.resnet20_ring8().replace(rounds=13),
    wl.vgg16_ring16(1).replace(rounds=7),             # layers on both paths: the side stream is part of the capture
    wl.vgg16_ring16(2).replace(rounds=6),             # the same at rank 2: two-column pair sweep beside the three sweeps
]


@pytest.mark.parametrize("w", REPLAY_CASES, ids=lambda w: w.name)
def test_pg_rounds_graph_replay_equals_repeated_pg_round_bit_for_bit(w):
    """Where pg_rounds replays a captured pair of rounds (static graph, steady state), the result
    is that of the same number of pg_round calls, whatever the split and the parity it starts from."""
    a, b = common.network_for(w), common.network_for(w)
    common.load_both(w, None, a)
    common.load_both(w, None, b)
    for _ in range(2 * w.rounds):
        a.pg_round()
    b.pg_rounds(w.rounds - 1)      # warm-up rounds one by one, then replays, then a remainder
    b.pg_round()                   # changes the parity the next replay starts from
    b.pg_rounds(w.rounds)
    assert a.pg_get_round() == b.pg_get_round() == 2 * w.rounds
    assert a.pg_kernel_launches() == b.pg_kernel_launches()
    assert a.pg_device_status() == 0 and b.pg_device_status() == 0
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            assert np.array_equal(a.pg_read_params(i, l), b.pg_read_params(i, l))
    e = a.pg_get_schedule(0)[0][0]
    assert np.array_equal(a.pg_read_q(int(e[0]), int(e[1]), 0), b.pg_read_q(int(e[0]), int(e[1]), 0))
    a.close()
    b.close()


@pytest.mark.parametrize("three_sweeps", [True, False], ids=["cooperative_kernel", "pair_sweep"])
def test_pg_rounds_against_the_checker(three_sweeps, monkeypatch):
    if three_sweeps:
        monkeypatch.setenv("PG_DISABLE_PAIR_SWEEP", "1")
    w = wl.tiny_ring()
    oracle, net = common.oracle_for(w), common.network_for(w)
    common.load_both(w, oracle, net)
    net.pg_rounds(w.rounds)
    oracle.round(w.rounds)
    err, where = common.max_relative_error(w, oracle, net)
    assert err <= REL_TOL, (err, where)
    net.close()
    oracle.close()


def test_grid_barrier_gives_up_instead_of_hanging():
    """A barrier that can never complete must time out, report it and leave the GPU usable."""
    from paper_2008_01425_b200 import binding as pg

    w = wl.tiny_ring()
    net = common.network_for(w)
    assert net.pg_selftest_barrier_timeout() == pg.PG_ERR_TIMEOUT
    # a context that saw a time-out runs no further round: its state may be mid-step
    for call in (net.pg_round, lambda: net.pg_rounds(3), lambda: net.pg_set_round(0)):
        with pytest.raises(pg.PowerGossipError) as e:
            call()
        assert e.value.status == pg.PG_ERR_STATE
    assert net.pg_device_status() == pg.PG_ERR_TIMEOUT          # sticky
    net.close()
    other = common.network_for(w)          # the device still works
    common.load_both(w, None, other)
    other.pg_rounds(2)
    assert other.pg_device_status() == pg.PG_OK
    other.close()


# ---- pair sweep on graphs of degree 2 (a row has two readers) ------------------
# thin rows (a warp per row), rows a CTA shares (TMA-fed up to 5120 floats, register-fed beyond),
# rows a cluster shares; few rows each, so the stack is small and every layer takes the pair sweep
DEGREE2_SHAPES = ((33, 130), (20, 1500), (40, 4612), (12, 6000), (9, 9000), (5, 3))
DEGREE2_GRAPHS = {
    "ring3": dict(n_workers=3, kind=wl.RING, custom_edges=()),
    "ring7": dict(n_workers=7, kind=wl.RING, custom_edges=()),
    "path5": dict(n_workers=5, kind=wl.CUSTOM, custom_edges=((0, 1), (1, 2), (2, 3), (3, 4))),
    "pair_and_path": dict(n_workers=5, kind=wl.CUSTOM, custom_edges=((0, 1), (2, 3), (3, 4))),
}


@pytest.mark.parametrize("graph", sorted(DEGREE2_GRAPHS))
def test_pair_sweep_on_graphs_of_degree_two(graph):
    # uniform weights 1/3: with Metropolis weights the isolated pair would get 1/2, which deflates its
    # difference exactly, and on these flat-spectrum matrices that makes the iteration follow rounding noise
    # (the checker alone, with X rounded to fp32 once per round, is then 3e-1 away after four rounds)
    w = wl.Workload("deg2_" + graph, 9, 4, wl.RING, 0, 0, wl.W_UNIFORM, None, DEGREE2_SHAPES, 1, 2, 6, 31,
                    "normal1").replace(**DEGREE2_GRAPHS[graph])
    _run(w, rebased=True)
    _run(w, rounds=3, check_every=1)


# rank 2 on graphs of degree 2: layers of at least 256 rows and 2^20 elements with rows of 1025..5120
# floats take the two-column CTA-per-row sweep (2, 3, 4 and 5 float4 per thread here), the rest the
# three sweeps on the side stream
RANK2_SHAPES = ((1024, 1100), (512, 2304), (300, 3600), (256, 4612), (40, 130))


@pytest.mark.parametrize("graph", ["ring3", "ring7", "path5", "pair_and_path"])
def test_rank_two_pair_sweep_on_graphs_of_degree_two(graph):
    w = wl.Workload("deg2_rank2_" + graph, 9, 4, wl.RING, 0, 0, wl.W_UNIFORM, None, RANK2_SHAPES, 2, 2, 4, 37,
                    "normal1").replace(**DEGREE2_GRAPHS[graph])
    _run(w, rebased=True)
    _run(w, rounds=3, check_every=1)


def test_rank_two_reads_between_steps_on_a_ring_run():
    """Reading after every round folds the pending rank-2 corrections into X, and the sweep that
    follows forms the difference from materialised rows instead of stored rows plus pending terms:
    the same numbers up to fp32 rounding (1e-6), and two reads in a row agree bit for bit."""
    w = wl.Workload("ring_reads_rank2", 9, 4, wl.RING, 0, 0, wl.W_UNIFORM, None, ((512, 2304), (24, 150)), 2, 1,
                    5, 3, "normal1")
    a, b = common.network_for(w), common.network_for(w)
    common.load_both(w, None, a)
    common.load_both(w, None, b)
    for t in range(w.rounds):
        a.pg_round()
        b.pg_round()
        first, again = b.read_all(), b.read_all()
        for i in range(w.n_workers):
            for l in range(2):
                assert np.array_equal(first[i][l], again[i][l])
    xa, xb = a.read_all(), b.read_all()
    for i in range(w.n_workers):
        for l in range(2):
            assert np.linalg.norm(xa[i][l] - xb[i][l]) <= 1e-6 * np.linalg.norm(xa[i][l])
    a.close()
    b.close()


def test_three_sweeps_on_a_rank_one_ring(monkeypatch):
    """The general path on a graph where the pair sweep is the default."""
    monkeypatch.setenv("PG_DISABLE_PAIR_SWEEP", "1")
    w = wl.Workload("ring_three_sweeps", 9, 6, wl.RING, 0, 0, wl.W_METROPOLIS, None, DEGREE2_SHAPES, 1, 2, 6, 31,
                    "normal1")
    _run(w, rebased=True)
    _run(wl.resnet20_ring8(), rounds=20, check_every=10)


def test_reads_between_steps_on_a_ring_run():
    """On a ring the corrected rows alternate between two copies of the stack and a read folds
    the pending correction into the first one.  At rank 1 the sweep that follows a read forms the
    difference from materialised rows, the one that follows another sweep from the rows as stored
    plus the pending terms as vector algebra: the same numbers up to fp32 rounding, so a run that
    is read (and check-pointed) after every round stays within 1e-6 of one that is never touched,
    and a read or a resume leaves the state itself untouched (two reads in a row agree bit for bit)."""
    w = wl.Workload("ring_reads", 9, 5, wl.RING, 0, 0, wl.W_UNIFORM, None, ((70, 130), (24, 1500)), 1, 1, 7, 3,
                    "normal1")
    a, b = common.network_for(w), common.network_for(w)
    common.load_both(w, None, a)
    common.load_both(w, None, b)
    for t in range(w.rounds):
        a.pg_round()
        b.pg_round()
        first = b.read_all()
        again = b.read_all()
        for i in range(w.n_workers):
            for l in range(2):
                assert np.array_equal(first[i][l], again[i][l])
    xa, xb = a.read_all(), b.read_all()
    # resume from a snapshot taken after an odd number of steps
    c = common.network_for(w)
    common.load_both(w, None, c)
    for t in range(3):
        c.pg_round()
    snap_x = c.read_all()
    edges = [(int(i), int(j)) for i, j in c.pg_get_schedule(0)[0]]
    snap_q = {(i, j): [c.pg_read_q(i, j, l) for l in range(2)] for i, j in edges}
    d = common.network_for(w)
    d.write_all(snap_x)
    for (i, j), qs in snap_q.items():
        for l, q in enumerate(qs):
            d.pg_write_q(i, j, l, q)
    d.pg_set_round(3)
    for t in range(3, w.rounds):
        c.pg_round()
        d.pg_round()
    xc, xd = c.read_all(), d.read_all()
    for i in range(w.n_workers):
        for l in range(2):
            scale = np.linalg.norm(xa[i][l])
            assert np.linalg.norm(xa[i][l] - xb[i][l]) <= 1e-6 * scale
            assert np.linalg.norm(xa[i][l] - xc[i][l]) <= 1e-6 * scale
            assert np.array_equal(xc[i][l], xd[i][l])      # the snapshot {X, Q, round} is the whole state
    for n in (a, b, c, d):
        n.close()


# ---- Algorithm 2 read literally (half-step mode) ------------------------------
def _run_half(w, rounds, rebase_every=None, check_every=1):
    """Half-step mode on both sides.  `power_steps` counts iterations per round.  Re-basing
    (checker state -> fp32 -> both sides) only happens after an even number of iterations,
    when the pair vectors are back in R^cols and can be written through pg_write_q."""
    from paper_2008_01425_b200 import binding as pg

    oracle, net = common.oracle_for(w), common.network_for(w)
    oracle.set_half_step()
    common.load_both(w, oracle, net)
    net.pg_set_half_step()
    avg0 = [common.initial_average(w, l) for l in range(len(w.layer_shapes))]
    pairs = set((int(a), int(b)) for a, b in oracle.round_schedule(0)[0])
    for t in range(1, rounds + 1):
        net.pg_round()
        oracle.round()
        if t % check_every == 0 or t == rounds:
            err, where = common.max_relative_error(w, oracle, net)     # reading X flushes a pending update
            assert err <= REL_TOL, "round %d: relative error %.3e at %r" % (t, err, where)
        if rebase_every and t % rebase_every == 0 and t < rounds:
            assert (t * w.power_steps) % 2 == 0
            common.rebase(w, oracle, net, pairs)
    assert net.pg_device_status() == pg.PG_OK
    _check_average(w, net, avg0)
    net.close()
    oracle.close()


def test_half_step_tiny_ring_free_running():
    _run_half(wl.tiny_ring(), 20, check_every=1)       # a read after every odd iteration: the flush path


def test_half_step_tiny_ring_few_reads():
    _run_half(wl.tiny_ring(), 20, check_every=20)      # pending updates consumed by the transposed sweep


def test_half_step_resnet20_two_iterations_rebased():
    _run_half(wl.resnet20_ring8().replace(power_steps=2), 30, rebase_every=4, check_every=2)


def test_half_step_torus_small_three_iterations_rebased():
    w = wl.shrink(wl.torus8x8(3), [(200, 136)], 12)
    _run_half(w, 12, rebase_every=2, check_every=1)


@pytest.mark.parametrize("iterations", [1, 2])
def test_half_step_ragged_shapes(iterations):
    w = wl.Workload("half_edge", 9, 4, wl.RING, 0, 0, wl.W_EXPLICIT, 0.3,
                    ((67, 131), (5, 3), (9, 1), (1, 9), (300, 7)), 1, iterations, 6, 77, "normal1")
    _run_half(w, 6, rebase_every=2)


def test_half_step_mode_is_refused_where_it_does_not_apply():
    from paper_2008_01425_b200 import binding as pg

    for w in (wl.tiny_ring().replace(rank=2), wl.shrink(wl.lstm_matching32(), [(30, 20)], 1).replace(n_workers=4)):
        net = common.network_for(w)
        with pytest.raises(pg.PowerGossipError) as e:
            net.pg_set_half_step()
        assert e.value.status == pg.PG_ERR_INVALID
        net.close()
    net = common.network_for(wl.tiny_ring())
    common.load_both(wl.tiny_ring(), None, net)
    net.pg_round()
    with pytest.raises(pg.PowerGossipError) as e:
        net.pg_set_half_step()
    assert e.value.status == pg.PG_ERR_STATE
    net.close()


# ---- Algorithm 1: a local gradient term between gossip rounds ----------------
@pytest.mark.parametrize("w", [wl.tiny_ring(), wl.shrink(wl.lstm_matching32(), [(130, 70), (70, 1300)], 6).replace(n_workers=8)],
                         ids=lambda w: w.name)
def test_local_gradient_steps_between_rounds(w):
    """X_i <- X_i + gossip - eta G with a synthetic per-worker G, applied by the caller
    in place through pg_params_device (torch) and by add_params on the checker."""
    import torch

    oracle, net = common.oracle_for(w), common.network_for(w)
    common.load_both(w, oracle, net)
    eta = 0.05
    for t in range(6):
        net.pg_round()
        oracle.round()
        for i in range(w.n_workers):
            for l, (n, m) in enumerate(w.layer_shapes):
                g = np.random.default_rng([t, i, l]).standard_normal((n, m)).astype(np.float32)
                view = net.pg_params_device(i, l)
                assert tuple(view.shape) == (n, m)
                view -= eta * torch.from_numpy(g).to(view.device)
                oracle.add_params(i, l, -(np.float64(np.float32(eta)) * g.astype(np.float64)))
        err, where = common.max_relative_error(w, oracle, net)
        assert err <= REL_TOL, (t, err, where)
    net.close()
    oracle.close()


SGD_CASES = {
    "ring_pair_sweep": (wl.tiny_ring().replace(layer_shapes=((64, 32), (9, 1500), (5, 3))), None),
    "ring_pair_sweep_two_steps": (wl.tiny_ring().replace(layer_shapes=((33, 130), (7, 9000)), power_steps=2), None),
    "matching_pair_sweep": (wl.shrink(wl.lstm_matching32(), [(130, 70), (70, 1300)], 6).replace(n_workers=8), None),
    "torus_rank2_two_steps": (wl.shrink(wl.torus8x8(2), [(200, 136), (5, 3)], 6).replace(rank=2), None),
    "ring_rank2_pair_sweep": (wl.tiny_ring().replace(layer_shapes=((512, 2306), (33, 130)), rank=2, power_steps=2), None),
    "ring_three_sweeps": (wl.tiny_ring().replace(layer_shapes=((64, 32), (67, 131))), "three"),
    "ring_half_step": (wl.tiny_ring().replace(power_steps=3), "half"),
    "ring_random_projection": (wl.tiny_ring().replace(rank=2), "random"),
}


@pytest.mark.parametrize("case", sorted(SGD_CASES))
def test_round_with_fused_gradient_step(case, monkeypatch):
    """pg_round_sgd: X <- X + gossip - eta G with G read by the sweep that applies the update
    (Algorithm 1, line 6).  The checker does the round, then add_params(-eta G) in fp64.  The
    padding columns of the gradient buffer are filled with NaN: they must not be read into X."""
    import torch

    w, mode = SGD_CASES[case]
    if mode == "three":
        monkeypatch.setenv("PG_DISABLE_PAIR_SWEEP", "1")
    oracle, net = common.oracle_for(w), common.network_for(w)
    if mode == "half":
        oracle.set_half_step()
    if mode == "random":
        oracle.set_random_projection(1)
    common.load_both(w, oracle, net)
    if mode == "half":
        net.pg_set_half_step()
    if mode == "random":
        net.pg_set_random_projection(1)
    grads = net.gradient_buffer()
    grads.fill_(float("nan"))
    eta = 0.05
    for t in range(5):
        for i in range(w.n_workers):
            for l, (n, m) in enumerate(w.layer_shapes):
                g = np.random.default_rng([t, i, l]).standard_normal((n, m)).astype(np.float32)
                net.gradient_view(grads, i, l).copy_(torch.from_numpy(g))
        net.pg_round_sgd(grads, eta)
        oracle.round()
        for i in range(w.n_workers):
            for l, (n, m) in enumerate(w.layer_shapes):
                g = np.random.default_rng([t, i, l]).standard_normal((n, m)).astype(np.float32)
                oracle.add_params(i, l, -(np.float64(np.float32(eta)) * g.astype(np.float64)))
        torch.cuda.synchronize()
        if t % 2 == 1 or t == 4:        # some rounds follow each other without a read in between
            err, where = common.max_relative_error(w, oracle, net)
            assert err <= REL_TOL, (t, err, where)
    assert net.pg_device_status() == 0
    assert net.pg_get_round() == 5
    net.close()
    oracle.close()


def test_round_with_gradient_rejects_bad_buffers():
    import torch
    from paper_2008_01425_b200 import binding as pg

    w = wl.tiny_ring()
    net = common.network_for(w)
    common.load_both(w, None, net)
    grads = net.gradient_buffer()
    assert grads.numel() == net.pg_stack_elems() and net.pg_stack_offset(1, 0)[0] % 64 == 0
    with pytest.raises(pg.PowerGossipError) as e:
        net.pg_round_sgd(grads, float("inf"))
    assert e.value.status == pg.PG_ERR_INVALID
    bigger = torch.zeros(grads.numel() + 8, dtype=torch.float32, device=grads.device)
    with pytest.raises(pg.PowerGossipError) as e:
        net.pg_round_sgd(bigger[1:], 0.1)          # 4-byte aligned only
    assert e.value.status == pg.PG_ERR_INVALID
    assert net.pg_get_round() == 0
    net.close()


# ---- random-projection compressors (Section 5.1) ------------------------------
RANDOM_CASES = [
    wl.tiny_ring().replace(rounds=30),
    wl.tiny_ring().replace(rounds=10, rank=4, power_steps=2),
    wl.resnet20_ring8().replace(rounds=20),
    wl.shrink(wl.torus8x8(2), [(200, 136)], 20).replace(rank=2),
    wl.Workload("rand_edge", 9, 4, wl.RING, 0, 0, wl.W_EXPLICIT, 0.3,
                ((67, 131), (5, 3), (9, 1), (1, 9), (3, 2500)), 2, 1, 8, 77, "normal1"),
]


@pytest.mark.parametrize("mode", [1, 2], ids=["right", "left"])
@pytest.mark.parametrize("w", RANDOM_CASES, ids=lambda w: "%s_r%d" % (w.name, w.rank))
def test_random_projection_compressors(w, mode):
    """The update is linear in X for given directions, so a free-running comparison over all
    rounds is meaningful here (no warm-started state, no chaos)."""
    from paper_2008_01425_b200 import binding as pg

    oracle, net = common.oracle_for(w), common.network_for(w)
    oracle.set_random_projection(mode)
    common.load_both(w, oracle, net)
    net.pg_set_random_projection(mode)
    avg0 = [common.initial_average(w, l) for l in range(len(w.layer_shapes))]
    for _ in range(w.rounds):
        net.pg_round()
    oracle.round(w.rounds)
    err, where = common.max_relative_error(w, oracle, net)
    assert err <= REL_TOL, (err, where)
    assert net.pg_device_status() == pg.PG_OK
    _check_average(w, net, avg0)
    d_ref, d_gpu = oracle.consensus_distance(), common.gpu_consensus_distance(w, net)
    assert abs(d_gpu - d_ref) <= 1e-3 * d_ref
    net.close()
    oracle.close()


def test_random_projection_is_refused_on_a_matching():
    from paper_2008_01425_b200 import binding as pg

    net = common.network_for(wl.shrink(wl.lstm_matching32(), [(30, 20)], 1).replace(n_workers=4))
    with pytest.raises(pg.PowerGossipError) as e:
        net.pg_set_random_projection(pg.PG_RANDOM_RIGHT)
    assert e.value.status == pg.PG_ERR_INVALID
    net.close()
