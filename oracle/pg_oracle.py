"""ctypes binding of the fp64 CPU checker in ``pg_oracle.c``.

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; the CUDA library and its Python
binding never do.  Every number it returns is computed by ``pg_oracle.c``;
this file only builds that C file with gcc, marshals arrays and owns handles.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# PG_ORACLE_SRC / PG_ORACLE_BUILD let the mutation tests point the binding at a
# deliberately broken copy of the C file (to show that the pins catch it).
_SRC = os.environ.get("PG_ORACLE_SRC", os.path.join(_HERE, "pg_oracle.c"))
_BUILD = os.environ.get("PG_ORACLE_BUILD", os.path.join(_HERE, "_build"))
_LIB = os.path.join(_BUILD, "libpg_oracle.so")

RING, TORUS, MATCHING, CUSTOM = 0, 1, 2, 3
W_UNIFORM, W_METROPOLIS, W_EXPLICIT = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile pg_oracle.c (gcc, -O2, OpenMP) into oracle/_build/."""
    os.makedirs(_BUILD, exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        c_int, c_u64, c_i64, c_dbl = ctypes.c_int, ctypes.c_uint64, ctypes.c_int64, ctypes.c_double
        vp = ctypes.c_void_p
        L.pgo_philox4x32_10.argtypes = [vp, vp, vp]
        L.pgo_philox4x32_10.restype = None
        L.pgo_init_q.argtypes = [c_u64, c_int, c_int, c_int, c_int, c_int, vp]
        L.pgo_init_q.restype = None
        L.pgo_schedule.argtypes = [c_int, c_int, c_int, c_int, vp, c_int, c_u64, c_i64, vp]
        L.pgo_schedule.restype = c_int
        L.pgo_edge_weights.argtypes = [c_int, c_int, vp, c_int, vp, c_int, vp]
        L.pgo_edge_weights.restype = c_int
        L.pgo_create.argtypes = [c_int, c_int, c_int, c_int, vp, c_int, c_int, vp, vp, c_int,
                                 c_int, c_int, c_u64]
        L.pgo_create.restype = vp
        L.pgo_destroy.argtypes = [vp]
        L.pgo_destroy.restype = None
        L.pgo_set_params.argtypes = [vp, c_int, c_int, vp]
        L.pgo_set_params.restype = c_int
        L.pgo_add_params.argtypes = [vp, c_int, c_int, vp]
        L.pgo_add_params.restype = c_int
        L.pgo_get_params.argtypes = [vp, c_int, c_int, vp]
        L.pgo_get_params.restype = c_int
        for f in (L.pgo_get_q, L.pgo_set_q, L.pgo_get_phat):
            f.argtypes = [vp, c_int, c_int, c_int, vp]
            f.restype = c_int
        L.pgo_get_round.argtypes = [vp]
        L.pgo_get_round.restype = c_i64
        L.pgo_set_round.argtypes = [vp, c_i64]
        L.pgo_set_round.restype = None
        L.pgo_round_schedule.argtypes = [vp, c_i64, vp, vp]
        L.pgo_round_schedule.restype = c_int
        L.pgo_round.argtypes = [vp]
        L.pgo_round.restype = c_int
        L.pgo_consensus_distance.argtypes = [vp]
        L.pgo_consensus_distance.restype = c_dbl
        L.pgo_average.argtypes = [vp, c_int, vp]
        L.pgo_average.restype = c_int
        L.pgo_compression_ratio.argtypes = [c_int, c_int, c_int, c_int]
        L.pgo_compression_ratio.restype = c_dbl
        L.pgo_set_random_projection.argtypes = [vp, c_int]
        L.pgo_set_random_projection.restype = c_int
        L.pgo_random_directions.argtypes = [c_u64, c_i64, c_int, c_int, c_int, c_int, c_int, vp]
        L.pgo_random_directions.restype = None
        L.pgo_set_half_step.argtypes = [vp, c_int]
        L.pgo_set_half_step.restype = c_int
        L.pgo_get_vector.argtypes = [vp, c_int, c_int, c_int, vp]
        L.pgo_get_vector.restype = c_int
        L.pgo_min_residual_ratio.argtypes = [vp]
        L.pgo_min_residual_ratio.restype = c_dbl
        L.pgo_set_fp32_storage.argtypes = [vp, c_int]
        L.pgo_set_fp32_storage.restype = c_int
        L.pgo_set_num_threads.argtypes = [c_int]
        L.pgo_set_num_threads.restype = None
        L.pgo_num_threads.argtypes = []
        L.pgo_num_threads.restype = c_int
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().pgo_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return tuple(int(v) for v in out)


def init_q(seed: int, i: int, j: int, layer: int, col: int, m: int) -> np.ndarray:
    out = np.zeros(m, dtype=np.float32)
    lib().pgo_init_q(seed, i, j, layer, col, m, _ptr(out))
    return out


def schedule(kind: int, n_workers: int, torus_rows: int = 0, torus_cols: int = 0,
             custom_edges: Sequence[Tuple[int, int]] = (), seed: int = 0,
             round_index: int = 0) -> np.ndarray:
    """Canonical edge list of one round as an (E, 2) int32 array."""
    cust = np.asarray(custom_edges, dtype=np.int32).reshape(-1, 2)
    cap = max(2 * n_workers, len(cust), 1)
    out = np.zeros((cap, 2), dtype=np.int32)
    E = lib().pgo_schedule(kind, n_workers, torus_rows, torus_cols,
                           _ptr(cust) if len(cust) else None, len(cust), seed, round_index,
                           _ptr(out))
    if E < 0:
        raise ValueError("invalid topology")
    return out[:E].copy()


def edge_weights(rule: int, n_workers: int, edges: np.ndarray,
                 W: Optional[np.ndarray] = None, allow_zero: bool = False) -> np.ndarray:
    edges = np.ascontiguousarray(edges, dtype=np.int32)
    Wf = None if W is None else np.ascontiguousarray(W, dtype=np.float32)
    out = np.zeros(len(edges), dtype=np.float64)
    rc = lib().pgo_edge_weights(rule, n_workers, _ptr(edges), len(edges), _ptr(Wf),
                                int(allow_zero), _ptr(out))
    if rc != 0:
        raise ValueError("mixing matrix violates Assumption A4")
    return out


def compression_ratio(n: int, m: int, rank: int = 1, iterations: int = 1) -> float:
    return float(lib().pgo_compression_ratio(n, m, rank, iterations))


def num_threads() -> int:
    return int(lib().pgo_num_threads())


def set_num_threads(n: int) -> None:
    """Threads the checker's parallel loops use from now on (timing only)."""
    lib().pgo_set_num_threads(int(n))


RANDOM_RIGHT, RANDOM_LEFT = 1, 2


def random_directions(seed: int, step: int, i: int, j: int, layer: int, length: int, rank: int) -> np.ndarray:
    """(length, rank) orthonormal directions of one pair, layer and step."""
    out = np.zeros((rank, length), dtype=np.float64)
    lib().pgo_random_directions(seed, step, i, j, layer, length, rank, _ptr(out))
    return out.T.copy()


class Oracle:
    """A whole simulated network in fp64 on the CPU."""

    def __init__(self, kind: int, n_workers: int, layer_shapes: Sequence[Tuple[int, int]],
                 rank: int = 1, power_steps: int = 1, seed: int = 0,
                 torus_rows: int = 0, torus_cols: int = 0,
                 custom_edges: Sequence[Tuple[int, int]] = (),
                 weight_rule: int = W_METROPOLIS, W: Optional[np.ndarray] = None):
        self.n_workers = int(n_workers)
        self.layer_shapes = [(int(a), int(b)) for a, b in layer_shapes]
        self.rank = int(rank)
        cust = np.asarray(custom_edges, dtype=np.int32).reshape(-1, 2)
        shapes = np.asarray(self.layer_shapes, dtype=np.int32).reshape(-1, 2)
        Wf = None if W is None else np.ascontiguousarray(W, dtype=np.float32)
        self._cap = max(2 * self.n_workers, len(cust), 1)
        self._h = lib().pgo_create(kind, self.n_workers, torus_rows, torus_cols,
                                   _ptr(cust) if len(cust) else None, len(cust),
                                   weight_rule, _ptr(Wf), _ptr(shapes), len(shapes),
                                   self.rank, int(power_steps), int(seed))
        if not self._h:
            raise ValueError("invalid topology, mixing matrix or sizes")

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().pgo_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def set_params(self, worker: int, layer: int, x: np.ndarray) -> None:
        x = np.ascontiguousarray(x, dtype=np.float32)
        assert x.shape == self.layer_shapes[layer]
        assert lib().pgo_set_params(self._h, worker, layer, _ptr(x)) == 0

    def add_params(self, worker: int, layer: int, delta: np.ndarray) -> None:
        """X_worker[layer] += delta in fp64 (Algorithm 1's -eta*G term)."""
        d = np.ascontiguousarray(delta, dtype=np.float64)
        assert d.shape == self.layer_shapes[layer]
        assert lib().pgo_add_params(self._h, worker, layer, _ptr(d)) == 0

    def get_params(self, worker: int, layer: int) -> np.ndarray:
        out = np.zeros(self.layer_shapes[layer], dtype=np.float64)
        assert lib().pgo_get_params(self._h, worker, layer, _ptr(out)) == 0
        return out

    def get_q(self, i: int, j: int, layer: int) -> np.ndarray:
        """(cols, rank) array: the pair's stored right factor."""
        m = self.layer_shapes[layer][1]
        out = np.zeros((self.rank, m), dtype=np.float64)
        assert lib().pgo_get_q(self._h, i, j, layer, _ptr(out)) == 0
        return out.T.copy()

    def set_q(self, i: int, j: int, layer: int, q: np.ndarray) -> None:
        m = self.layer_shapes[layer][1]
        q = np.asarray(q, dtype=np.float64).reshape(m, self.rank)
        src = np.ascontiguousarray(q.T)
        assert lib().pgo_set_q(self._h, i, j, layer, _ptr(src)) == 0

    def get_phat(self, i: int, j: int, layer: int) -> np.ndarray:
        """(rows, rank) array: the pair's last orthonormal left factor."""
        n = self.layer_shapes[layer][0]
        out = np.zeros((self.rank, n), dtype=np.float64)
        if lib().pgo_get_phat(self._h, i, j, layer, _ptr(out)) != 0:
            raise KeyError("pair has not been an edge yet")
        return out.T.copy()

    def set_random_projection(self, mode: int) -> None:
        """RANDOM_RIGHT: C(X) = (X U) U^T;  RANDOM_LEFT: C(X) = V (V^T X); fresh orthonormal
        directions per edge, layer and step (0 switches back to power iteration)."""
        if lib().pgo_set_random_projection(self._h, int(mode)) != 0:
            raise ValueError("random projections must be chosen before the first round")

    def set_half_step(self, on: bool = True) -> None:
        """Algorithm 2 read literally: one mat-vec and one update per iteration;
        `power_steps` then counts iterations per round.  Rank 1, static graphs."""
        if lib().pgo_set_half_step(self._h, int(on)) != 0:
            raise ValueError("half-step mode needs rank 1, a static graph and round 0")

    def min_residual_ratio(self) -> float:
        """Smallest squared (Gram-Schmidt residual / column before projection) met so far at a
        column k > 0 (inf if none): what the dependent-column rule compares with 1e-10."""
        return float(lib().pgo_min_residual_ratio(self._h))

    def set_fp32_storage(self, on: bool = True) -> None:
        """Test aid, not the method: round X and the touched vectors to fp32 after every power
        step (arithmetic stays fp64), the least perturbation an fp32-storage implementation applies."""
        if lib().pgo_set_fp32_storage(self._h, int(on)) != 0:
            raise ValueError("fp32 storage emulation is for power-iteration mode only")

    def get_vector(self, i: int, j: int, layer: int) -> np.ndarray:
        """The pair's current vector (rows entries after an odd iteration, else cols)."""
        n, m = self.layer_shapes[layer]
        out = np.zeros(max(n, m), dtype=np.float64)
        k = lib().pgo_get_vector(self._h, i, j, layer, _ptr(out))
        assert k > 0
        return out[:k].copy()

    @property
    def round_index(self) -> int:
        return int(lib().pgo_get_round(self._h))

    @round_index.setter
    def round_index(self, r: int) -> None:
        lib().pgo_set_round(self._h, int(r))

    def round_schedule(self, round_index: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
        r = self.round_index if round_index is None else int(round_index)
        edges = np.zeros((self._cap, 2), dtype=np.int32)
        w = np.zeros(self._cap, dtype=np.float64)
        E = lib().pgo_round_schedule(self._h, r, _ptr(edges), _ptr(w))
        if E < 0:
            raise ValueError("invalid schedule")
        return edges[:E].copy(), w[:E].copy()

    def round(self, n: int = 1) -> None:
        for _ in range(n):
            if lib().pgo_round(self._h) != 0:
                raise RuntimeError("oracle round failed")

    def consensus_distance(self) -> float:
        return float(lib().pgo_consensus_distance(self._h))

    def average(self, layer: int) -> np.ndarray:
        out = np.zeros(self.layer_shapes[layer], dtype=np.float64)
        assert lib().pgo_average(self._h, layer, _ptr(out)) == 0
        return out

    def all_params(self) -> List[List[np.ndarray]]:
        return [[self.get_params(i, l) for l in range(len(self.layer_shapes))]
                for i in range(self.n_workers)]
