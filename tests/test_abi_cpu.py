"""CPU-only checks of the C ABI: the library loads, exports every symbol the
header declares, validates its arguments, and its host-side schedule builder
and seeding agree bit for bit with the CPU checker's independent ones."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import pg_oracle as po
from paper_2008_01425_b200 import binding as pg
from paper_2008_01425_b200 import build as pg_build
from paper_2008_01425_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    pg_build.build()


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"PG_API[^;(]*?\b(pg_[a-z_0-9]+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert len(names) >= 15
    lib = ctypes.CDLL(pg.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(pg.EXPORTS)


def test_status_strings():
    assert pg.pg_status_string(pg.PG_OK) == "ok"
    seen = {pg.pg_status_string(s) for s in range(7)}
    assert len(seen) == 7


def test_workspace_bytes_and_argument_checks():
    b1 = pg.pg_workspace_bytes(pg.PG_RING, 4, [(64, 32)], 1)
    b2 = pg.pg_workspace_bytes(pg.PG_RING, 8, [(64, 32)], 1)
    assert 4 * 64 * 32 * 4 < b1 < b2
    lstm = wl.lstm_matching32()
    big = pg.pg_workspace_bytes(lstm.kind, lstm.n_workers, lstm.layer_shapes, lstm.rank)
    assert 4 * lstm.total_params < big < 4 * lstm.total_params * 1.05   # vectors and tables are ~1-2 %
    for bad in (dict(kind=pg.PG_MATCHING, n_workers=7), dict(kind=pg.PG_TORUS, n_workers=10, torus_rows=3, torus_cols=3),
                dict(kind=pg.PG_RING, n_workers=1), dict(kind=9, n_workers=4)):
        with pytest.raises(pg.PowerGossipError) as e:
            pg.pg_workspace_bytes(layer_shapes=[(8, 8)], rank=1, **bad)
        assert e.value.status == pg.PG_ERR_INVALID
    with pytest.raises(pg.PowerGossipError):
        pg.pg_workspace_bytes(pg.PG_RING, 4, [(8, 8)], 5)            # rank above the limit
    with pytest.raises(pg.PowerGossipError):
        pg.pg_workspace_bytes(pg.PG_TORUS, 16, [(8, 8)], 4, 4, 4)    # degree 4 x rank 4 vectors
    with pytest.raises(pg.PowerGossipError):
        pg.pg_workspace_bytes(pg.PG_RING, 4, [(0, 8)], 1)


def test_create_rejects_a_missing_workspace_without_touching_a_gpu():
    lib = pg.load_library()
    topo, keep = pg._topology(pg.PG_RING, 4, 0, 0, pg.PG_W_UNIFORM, ())
    h = ctypes.c_void_p()
    rc = lib.pg_create(ctypes.byref(topo), None, pg._shapes([(8, 8)]), 1, 1, 1, 0, None, 0, ctypes.byref(h))
    assert rc == pg.PG_ERR_WORKSPACE
    rc = lib.pg_create(ctypes.byref(topo), None, pg._shapes([(8, 8)]), 1, 1, 0, 0, None, 0, ctypes.byref(h))
    assert rc == pg.PG_ERR_INVALID                                    # power_steps < 1
    lib.pg_destroy(None)


SCHEDULE_CASES = [
    dict(kind=0, n_workers=2), dict(kind=0, n_workers=3), dict(kind=0, n_workers=8), dict(kind=0, n_workers=16),
    dict(kind=1, n_workers=64, torus_rows=8, torus_cols=8), dict(kind=1, n_workers=8, torus_rows=2, torus_cols=4),
    dict(kind=1, n_workers=6, torus_rows=1, torus_cols=6), dict(kind=1, n_workers=12, torus_rows=3, torus_cols=4),
    dict(kind=3, n_workers=6, custom_edges=[(5, 0), (0, 1), (1, 0), (2, 2), (3, 1), (4, 3)]),
]


@pytest.mark.parametrize("case", SCHEDULE_CASES)
@pytest.mark.parametrize("rule", [pg.PG_W_UNIFORM, pg.PG_W_METROPOLIS])
def test_static_schedules_match_the_checker_bit_for_bit(case, rule):
    e_lib, w_lib = pg.pg_build_schedule(weight_rule=rule, **case)
    e_ref = po.schedule(case["kind"], case["n_workers"], case.get("torus_rows", 0), case.get("torus_cols", 0),
                        case.get("custom_edges", ()))
    assert e_lib.dtype == e_ref.dtype and np.array_equal(e_lib, e_ref)
    w_ref = po.edge_weights(rule, case["n_workers"], e_ref)
    assert np.array_equal(w_lib, w_ref.astype(np.float32))


def test_matching_schedules_match_the_checker_bit_for_bit():
    for N in (2, 4, 32, 64):
        for seed in (0, 1005, 2 ** 40 + 7):
            for t in list(range(25)) + [2 ** 33 + 5]:
                e_lib, w_lib = pg.pg_build_schedule(pg.PG_MATCHING, N, seed=seed, round_index=t)
                assert np.array_equal(e_lib, po.schedule(po.MATCHING, N, seed=seed, round_index=t))
                assert np.all(w_lib == np.float32(0.5))


def test_explicit_mixing_matrices():
    for w in (wl.tiny_ring(), wl.resnet20_ring8(), wl.vgg16_ring16()):
        W = wl.mixing_matrix(w)
        e_lib, w_lib = pg.pg_build_schedule(w.kind, w.n_workers, weight_rule=w.weight_rule, W=W)
        e_ref = po.schedule(w.kind, w.n_workers)
        assert np.array_equal(e_lib, e_ref)
        assert np.array_equal(w_lib, po.edge_weights(po.W_EXPLICIT, w.n_workers, e_ref, W).astype(np.float32))
    bad = wl.mixing_matrix(wl.tiny_ring()).copy()
    bad[0, 1] += 0.1
    with pytest.raises(pg.PowerGossipError):
        pg.pg_build_schedule(pg.PG_RING, 4, weight_rule=pg.PG_W_EXPLICIT, W=bad)
    with pytest.raises(pg.PowerGossipError):
        pg.pg_build_schedule(pg.PG_RING, 4, weight_rule=pg.PG_W_EXPLICIT, W=None)
    # a zero edge weight freezes an edge; only custom graphs accept it
    Wz = np.eye(2, dtype=np.float32)
    e, w = pg.pg_build_schedule(pg.PG_CUSTOM, 2, weight_rule=pg.PG_W_EXPLICIT, W=Wz, custom_edges=[(0, 1)])
    assert len(e) == 1 and w[0] == 0.0
    with pytest.raises(pg.PowerGossipError):
        pg.pg_build_schedule(pg.PG_RING, 2, weight_rule=pg.PG_W_EXPLICIT, W=Wz)


def test_initial_vectors_match_the_checker_bit_for_bit():
    for (seed, i, j, layer, col, m) in [(0, 0, 1, 0, 0, 1), (1005, 3, 17, 7, 0, 28000), (1004, 0, 15, 12, 1, 4608),
                                         (2 ** 63 + 11, 30, 31, 2, 3, 651), (1, 0, 1, 0, 0, 27)]:
        assert np.array_equal(pg.pg_initial_vector(seed, i, j, layer, col, m), po.init_q(seed, i, j, layer, col, m))


# --------------------------------------------------------------------------
# communication volume (host-only call)
# --------------------------------------------------------------------------
def _golden(name):
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_comm_floats_reproduce_the_printed_per_tensor_ratios():
    """Appendix, parameter tables: rank-1 PowerGossip with r iterations compresses an
    n x m tensor n*m / ((n+m)/2) / r times; the tables print that ratio rounded ("115/r x")."""
    for n, m, printed in _golden("compression_ratios.txt"):
        n, m, printed = int(n), int(m), int(printed)
        two, dense = pg.pg_comm_floats([(n, m)], 1, 1, 2)           # an odd and an even iteration
        assert dense == n * m and two == n + m
        assert round(dense / (two / 2)) == printed
        odd, _ = pg.pg_comm_floats([(n, m)], 1, 1, 1)
        even, _ = pg.pg_comm_floats([(n, m)], 1, 2, 1)
        assert (odd, even) == (n, m)                                 # p has `rows` entries, the transposed step `cols`
        assert pg.pg_comm_floats([(n, m)], 3, 4, 5)[0] == 3 * (2 * n + 3 * m)   # k = 4..8: three even, two odd
    with pytest.raises(pg.PowerGossipError):
        pg.pg_comm_floats([(4, 4)], 1, 0, 1)


def test_comm_floats_reproduce_the_printed_whole_model_ratios():
    """Result tables: bytes sent per epoch of PowerGossip against D-PSGD.  Every message carries
    the matrices' vectors plus the 1-D tensors uncompressed, so the ratio is
    (dense + bias) / (iterations x mean floats per iteration + bias)."""
    lstm_paper = ((28869, 650),) + ((2600, 650),) * 6      # the paper's own LSTM table (tied decoder)
    for model, iterations, printed, bias_bytes in _golden("comm_volume.txt"):
        shapes = wl.RESNET20_SHAPES if model == "resnet20" else lstm_paper
        iterations, printed, bias_bytes = int(iterations), int(printed), int(bias_bytes)
        two, dense = pg.pg_comm_floats(shapes, 1, 1, 2)
        sent_bytes = 4.0 * iterations * two / 2 + bias_bytes
        ratio = (4.0 * dense + bias_bytes) / sent_bytes
        if model == "resnet20":
            assert round(ratio) == printed, (model, iterations, ratio)
        else:
            assert abs(ratio / printed - 1.0) < 0.025, (model, iterations, ratio)
