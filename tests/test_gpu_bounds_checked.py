"""The bounds-checked build of the library (-DPG_BOUNDS_CHECK), the stand-in for a memory checker.

Every kernel of that build verifies the address ranges it is about to touch against the section
of the workspace they belong to; an address outside raises PG_ERR_BOUNDS in the status word and the
access is skipped.  Here the checked library runs, in a process of its own, ragged shapes, graphs of
degree two at rank 1 and 2, the torus, a time-varying matching, the modes of Algorithm 2 read
literally and of the random projections, and one round of every full-size workload: the status word
must stay clean and the results must be the bits the regular build produces.
"""
import hashlib
import json
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2008_01425_b200 import workloads as wl

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import hashlib, json, sys
import numpy as np
sys.path.insert(0, %(root)r)
from paper_2008_01425_b200 import workloads as wl
from tests import common
from tests.test_gpu_bounds_checked import cases

out = {}
for name, w, rounds, mode in cases():
    net = common.network_for(w)
    common.load_both(w, None, net)
    if mode == "half":
        net.pg_set_half_step()
    if mode == "random":
        net.pg_set_random_projection(1)
    for _ in range(rounds):
        net.pg_round()
    h = hashlib.sha256()
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            h.update(net.pg_read_params(i, l).tobytes())
    out[name] = [net.pg_device_status(), h.hexdigest()]
    net.close()
probe = common.network_for(wl.tiny_ring())
out["__probe__"] = [probe.pg_selftest_bounds_check(), ""]
probe.close()
print("RESULT " + json.dumps(out))
"""


def cases():
    """(name, workload, rounds, mode)"""
    ragged = ((67, 131), (5, 3), (9, 1), (1, 9), (300, 7), (7, 2500))
    deg2 = ((33, 130), (20, 1500), (40, 4612), (12, 6000), (9, 9000), (5, 3))
    rank2 = ((1024, 1100), (512, 2304), (300, 3600), (256, 4612), (40, 130))
    ring = wl.Workload("c", 9, 5, wl.RING, 0, 0, wl.W_UNIFORM, None, ragged, 1, 2, 3, 77, "normal1")
    yield "ragged_ring_rank1", ring, 3, None
    yield "ragged_ring_rank4", ring.replace(rank=4), 2, None
    yield "degree2_ring7", ring.replace(n_workers=7, layer_shapes=deg2), 3, None
    yield "degree2_path", ring.replace(kind=wl.CUSTOM, custom_edges=((0, 1), (1, 2), (2, 3), (3, 4)), layer_shapes=deg2), 3, None
    yield "rank2_ring3", ring.replace(n_workers=3, rank=2, layer_shapes=rank2), 3, None
    yield "rank2_path", ring.replace(kind=wl.CUSTOM, custom_edges=((0, 1), (1, 2), (2, 3), (3, 4)), rank=2,
                                     layer_shapes=rank2), 2, None
    yield "torus_rank2", wl.shrink(wl.torus8x8(2), [(200, 136), (5, 3)], 3).replace(rank=2), 3, None
    yield "matching", wl.shrink(wl.lstm_matching32(), [(130, 70), (70, 1300), (9, 9000)], 4).replace(n_workers=8), 4, None
    yield "half_step", ring.replace(power_steps=3), 3, "half"
    yield "random_projection", ring.replace(rank=2), 3, "random"
    for w in (wl.tiny_ring(), wl.resnet20_ring8(), wl.torus8x8(2), wl.vgg16_ring16(1), wl.vgg16_ring16(2),
              wl.lstm_matching32()):
        yield "full_" + w.name + "_r%d" % w.rank, w, 2 if w.total_params < 1e9 else 1, None


def _run_child(library):
    env = dict(os.environ)
    if library:
        env["PG_LIBRARY"] = library
    else:
        env.pop("PG_LIBRARY", None)
    r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], cwd=ROOT, env=env, stdout=subprocess.PIPE,
                       stderr=subprocess.STDOUT, timeout=1500)
    text = r.stdout.decode()
    assert r.returncode == 0, text[-3000:]
    line = [l for l in text.splitlines() if l.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


def test_checked_build_is_clean_and_gives_the_same_bits():
    from paper_2008_01425_b200 import build as pg_build

    checked = pg_build.build(checked=True)
    got = _run_child(checked)
    want = _run_child(None)
    assert sorted(got) == sorted(want) and len(got) >= 17
    # the checks are really there: a range that ends one float past its section is reported, nothing else
    assert got.pop("__probe__")[0] == 8 and want.pop("__probe__")[0] == 0        # PG_ERR_BOUNDS, PG_OK
    for name in sorted(got):
        assert got[name][0] == 0, "%s: status %d in the checked build" % (name, got[name][0])
        assert want[name][0] == 0
        assert got[name][1] == want[name][1], "%s: the checked build gives other bits" % name
