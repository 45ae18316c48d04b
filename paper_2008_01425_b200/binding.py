"""Python binding of the C ABI in ``include/powergossip.h`` (ctypes).

Argument marshalling only: every step of a gossip round runs in the CUDA
kernels of ``libpowergossip.so``.  PyTorch is used for device memory (the
workspace tensor), pinned host buffers and streams.  There is no CPU fallback:
if the library has not been built, loading it raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# PG_LIBRARY selects another build of the same library (the bounds-checked one, see build.py)
LIB_PATH = os.environ.get("PG_LIBRARY") or os.path.join(_HERE, "libpowergossip.so")

(PG_OK, PG_ERR_INVALID, PG_ERR_WORKSPACE, PG_ERR_CUDA, PG_ERR_STATE, PG_ERR_TIMEOUT, PG_ERR_NUMERIC, PG_ERR_TOO_LARGE,
 PG_ERR_BOUNDS) = range(9)
PG_NOALLOC_MAX_PARTIALS = 1 << 20
PG_RING, PG_TORUS, PG_MATCHING, PG_CUSTOM = 0, 1, 2, 3
PG_W_UNIFORM, PG_W_METROPOLIS, PG_W_EXPLICIT = 0, 1, 2

EXPORTS = (
    "pg_workspace_bytes", "pg_create", "pg_destroy", "pg_write_params", "pg_read_params", "pg_read_params_async",
    "pg_round", "pg_device_status", "pg_get_schedule", "pg_max_edges", "pg_read_q", "pg_write_q",
    "pg_get_round", "pg_set_round", "pg_kernel_launches", "pg_status_string",
    "pg_build_schedule", "pg_initial_vector", "pg_timing_enable", "pg_timing_read",
    "pg_transposed_product_noalloc", "pg_rounds", "pg_selftest_barrier_timeout",
    "pg_set_half_step", "pg_params_device", "pg_set_random_projection",
    "pg_round_sgd", "pg_stack_elems", "pg_stack_offset", "pg_comm_floats", "pg_comm_floats_round",
    "pg_round_bytes", "pg_selftest_bounds_check",
)
PG_POWER_ITERATION, PG_RANDOM_RIGHT, PG_RANDOM_LEFT = 0, 1, 2
KERNEL_KINDS = ("forward", "edge_left", "transposed", "edge_right", "update_forward",
                "pair_sweep", "pair_edge", "update_only")


class pg_topology(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("n_workers", ctypes.c_int32),
                ("torus_rows", ctypes.c_int32), ("torus_cols", ctypes.c_int32),
                ("weight_rule", ctypes.c_int32), ("n_custom_edges", ctypes.c_int32),
                ("custom_edges", ctypes.POINTER(ctypes.c_int32))]


class pg_layer_shape(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int32), ("cols", ctypes.c_int32)]


class PowerGossipError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, pg_status_string(status), status))


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """Load libpowergossip.so; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2008_01425_b200.build` "
                          "(there is no CPU fallback)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64
    szp = ctypes.POINTER(ctypes.c_size_t)
    L.pg_workspace_bytes.argtypes = [ctypes.POINTER(pg_topology), ctypes.POINTER(pg_layer_shape), i32, i32, szp]
    L.pg_create.argtypes = [ctypes.POINTER(pg_topology), vp, ctypes.POINTER(pg_layer_shape), i32, i32, i32,
                            u64, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    L.pg_destroy.argtypes = [vp]
    L.pg_destroy.restype = None
    L.pg_write_params.argtypes = [vp, i32, i32, vp, vp]
    L.pg_read_params.argtypes = [vp, i32, i32, vp, vp]
    L.pg_read_params_async.argtypes = [vp, i32, i32, vp, vp]
    L.pg_round.argtypes = [vp, vp]
    L.pg_round_sgd.argtypes = [vp, vp, ctypes.c_float, vp]
    L.pg_stack_elems.argtypes = [vp, ctypes.POINTER(i64)]
    L.pg_stack_offset.argtypes = [vp, i32, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.pg_params_device.argtypes = [vp, i32, i32, vp, ctypes.POINTER(vp), ctypes.POINTER(i64)]
    L.pg_device_status.argtypes = [vp, vp]
    L.pg_rounds.argtypes = [vp, i32, vp]
    L.pg_set_half_step.argtypes = [vp, i32]
    L.pg_set_random_projection.argtypes = [vp, i32]
    L.pg_selftest_barrier_timeout.argtypes = [vp, vp]
    L.pg_selftest_bounds_check.argtypes = [vp, vp]
    L.pg_get_schedule.argtypes = [vp, i64, vp, vp, ctypes.POINTER(i32)]
    L.pg_max_edges.argtypes = [vp, ctypes.POINTER(i32)]
    L.pg_read_q.argtypes = [vp, i32, i32, i32, vp, vp]
    L.pg_write_q.argtypes = [vp, i32, i32, i32, vp, vp]
    L.pg_get_round.argtypes = [vp, ctypes.POINTER(i64)]
    L.pg_set_round.argtypes = [vp, i64, vp]
    L.pg_kernel_launches.argtypes = [vp, ctypes.POINTER(i64)]
    L.pg_build_schedule.argtypes = [ctypes.POINTER(pg_topology), vp, u64, i64, vp, vp, i32, ctypes.POINTER(i32)]
    L.pg_initial_vector.argtypes = [u64, i32, i32, i32, i32, i32, vp]
    L.pg_timing_enable.argtypes = [vp, i32]
    L.pg_timing_read.argtypes = [vp, vp, vp, vp]
    L.pg_transposed_product_noalloc.argtypes = [vp, i32, i32, i64, vp, vp, vp]
    L.pg_comm_floats.argtypes = [ctypes.POINTER(pg_layer_shape), i32, i32, i64, i64, ctypes.POINTER(i64),
                                 ctypes.POINTER(i64)]
    L.pg_comm_floats_round.argtypes = [vp, i64, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.pg_round_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.pg_status_string.argtypes = [ctypes.c_int]
    L.pg_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("pg_destroy", "pg_status_string"):
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def pg_status_string(status: int) -> str:
    return load_library().pg_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != PG_OK:
        raise PowerGossipError(status, where)


def _topology(kind, n_workers, torus_rows, torus_cols, weight_rule, custom_edges):
    edges = np.ascontiguousarray(np.asarray(custom_edges, dtype=np.int32).reshape(-1, 2))
    topo = pg_topology(kind, n_workers, torus_rows, torus_cols, weight_rule, len(edges),
                       edges.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)) if len(edges) else None)
    return topo, edges   # keep `edges` alive while `topo` is in use


def _shapes(layer_shapes):
    arr = (pg_layer_shape * len(layer_shapes))()
    for t, (n, m) in enumerate(layer_shapes):
        arr[t].rows, arr[t].cols = int(n), int(m)
    return arr


def pg_workspace_bytes(kind: int, n_workers: int, layer_shapes: Sequence[Tuple[int, int]], rank: int,
                       torus_rows: int = 0, torus_cols: int = 0, weight_rule: int = PG_W_METROPOLIS,
                       custom_edges: Sequence[Tuple[int, int]] = ()) -> int:
    topo, _keep = _topology(kind, n_workers, torus_rows, torus_cols, weight_rule, custom_edges)
    out = ctypes.c_size_t(0)
    _check(load_library().pg_workspace_bytes(ctypes.byref(topo), _shapes(layer_shapes), len(layer_shapes),
                                             rank, ctypes.byref(out)), "pg_workspace_bytes")
    return int(out.value)


def pg_build_schedule(kind: int, n_workers: int, seed: int = 0, round_index: int = 0,
                      torus_rows: int = 0, torus_cols: int = 0, weight_rule: int = PG_W_METROPOLIS,
                      custom_edges: Sequence[Tuple[int, int]] = (),
                      W: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Edge list (E, 2) int32 and weights (E,) fp32 of one round; host only, no GPU needed."""
    topo, keep = _topology(kind, n_workers, torus_rows, torus_cols, weight_rule, custom_edges)
    cap = max(2 * n_workers, len(keep), 1)
    edges = np.zeros((cap, 2), dtype=np.int32)
    w = np.zeros(cap, dtype=np.float32)
    n = ctypes.c_int32(0)
    Wf = None if W is None else np.ascontiguousarray(W, dtype=np.float32)
    _check(load_library().pg_build_schedule(ctypes.byref(topo), None if Wf is None else Wf.ctypes.data,
                                            seed, round_index, edges.ctypes.data, w.ctypes.data, cap,
                                            ctypes.byref(n)), "pg_build_schedule")
    return edges[:n.value].copy(), w[:n.value].copy()


def pg_initial_vector(seed: int, i: int, j: int, layer: int, col: int, m: int) -> np.ndarray:
    """Column `col` of the seeded initial vector of pair (i<j), layer `layer`; host only."""
    out = np.zeros(m, dtype=np.float32)
    _check(load_library().pg_initial_vector(seed, i, j, layer, col, m, out.ctypes.data), "pg_initial_vector")
    return out


def pg_comm_floats(layer_shapes: Sequence[Tuple[int, int]], rank: int = 1, first_iteration: int = 1,
                   iterations: int = 1) -> Tuple[int, int]:
    """(floats one end of one edge sends over these iterations of Algorithm 2, floats of one
    uncompressed exchange), summed over the layers; host only."""
    sent, dense = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(load_library().pg_comm_floats(_shapes(layer_shapes), len(layer_shapes), rank, first_iteration,
                                         iterations, ctypes.byref(sent), ctypes.byref(dense)), "pg_comm_floats")
    return int(sent.value), int(dense.value)


def pg_transposed_product_noalloc(X, p, z, stream=None, rows: Optional[int] = None,
                                  cols: Optional[int] = None, ld: Optional[int] = None) -> None:
    """z = X^T p on the GPU with the library's fixed scratch (no allocation).

    X: CUDA float32 tensor (rows x cols view; a row stride > cols is allowed),
    p: CUDA float32 vector of `rows` entries, z: CUDA float32 vector of `cols`
    entries, written in place.  Raises PowerGossipError(PG_ERR_TOO_LARGE) beyond
    the size limit stated in the header.
    """
    rows = int(X.shape[0]) if rows is None else rows
    cols = int(X.shape[1]) if cols is None else cols
    ld = int(X.stride(0)) if ld is None else ld
    _check(load_library().pg_transposed_product_noalloc(X.data_ptr(), rows, cols, ld, p.data_ptr(),
                                                        z.data_ptr(), _stream_handle(stream)),
           "pg_transposed_product_noalloc")


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream) or None


class PowerGossip:
    """One simulated network on one GPU (thin handle around ``pg_ctx``).

    The workspace is a ``torch.uint8`` tensor on ``device`` that this object
    keeps alive; every method forwards to the C function of the same name.
    """

    def __init__(self, kind: int, n_workers: int, layer_shapes: Sequence[Tuple[int, int]],
                 rank: int = 1, power_steps: int = 1, seed: int = 0,
                 torus_rows: int = 0, torus_cols: int = 0,
                 custom_edges: Sequence[Tuple[int, int]] = (),
                 weight_rule: int = PG_W_METROPOLIS, W: Optional[np.ndarray] = None,
                 device: str = "cuda:0", workspace=None):
        import torch

        self._lib = load_library()
        self._h = None
        self.n_workers = int(n_workers)
        self.layer_shapes = [(int(a), int(b)) for a, b in layer_shapes]
        self.rank = int(rank)
        self.power_steps = int(power_steps)
        self.device = torch.device(device)
        topo, _keep = _topology(kind, n_workers, torus_rows, torus_cols, weight_rule, custom_edges)
        shapes = _shapes(self.layer_shapes)
        nbytes = ctypes.c_size_t(0)
        _check(self._lib.pg_workspace_bytes(ctypes.byref(topo), shapes, len(self.layer_shapes), rank,
                                            ctypes.byref(nbytes)), "pg_workspace_bytes")
        self.workspace_bytes = int(nbytes.value)
        torch.cuda.set_device(self.device)
        if workspace is None:
            workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
        self._workspace = workspace
        base = workspace.data_ptr()
        aligned = (base + 255) // 256 * 256
        avail = workspace.numel() - (aligned - base)
        Wf = None if W is None else np.ascontiguousarray(W, dtype=np.float32)
        h = ctypes.c_void_p()
        _check(self._lib.pg_create(ctypes.byref(topo), None if Wf is None else Wf.ctypes.data,
                                   shapes, len(self.layer_shapes), rank, power_steps, seed,
                                   ctypes.c_void_p(aligned), avail, ctypes.byref(h)), "pg_create")
        self._h = h

    # -- lifetime ---------------------------------------------------------
    def pg_destroy(self) -> None:
        if self._h is not None:
            self._lib.pg_destroy(self._h)
            self._h = None

    close = pg_destroy

    def __del__(self):
        try:
            self.pg_destroy()
        except Exception:
            pass

    # -- parameters -------------------------------------------------------
    def pg_write_params(self, worker: int, layer: int, x, stream=None) -> None:
        """x: numpy array or CPU torch tensor, fp32, dense rows x cols."""
        ptr, _keep = _host_ptr(x, self.layer_shapes[layer])
        _check(self._lib.pg_write_params(self._h, worker, layer, ptr, _stream_handle(stream)),
               "pg_write_params")

    def pg_read_params(self, worker: int, layer: int, out=None, stream=None):
        if out is None:
            out = np.empty(self.layer_shapes[layer], dtype=np.float32)
        ptr, _keep = _host_ptr(out, self.layer_shapes[layer])
        _check(self._lib.pg_read_params(self._h, worker, layer, ptr, _stream_handle(stream)),
               "pg_read_params")
        return out

    def pg_read_params_async(self, worker: int, layer: int, out, stream=None):
        """Enqueue the copy into `out` (pinned CPU tensor or array) and return at once."""
        ptr, _keep = _host_ptr(out, self.layer_shapes[layer])
        _check(self._lib.pg_read_params_async(self._h, worker, layer, ptr, _stream_handle(stream)),
               "pg_read_params_async")
        return out

    def pg_params_device(self, worker: int, layer: int, stream=None):
        """(rows x cols) torch view of the worker's matrix in the workspace (row stride = the
        padded leading dimension), for in-place local updates such as  X -= eta * G."""
        import torch

        ptr, ld = ctypes.c_void_p(), ctypes.c_int64(0)
        _check(self._lib.pg_params_device(self._h, worker, layer, _stream_handle(stream), ctypes.byref(ptr),
                                          ctypes.byref(ld)), "pg_params_device")
        n, m = self.layer_shapes[layer]
        offset = (ptr.value - self._workspace.data_ptr()) // 4
        flat = self._workspace.view(torch.float32) if self._workspace.data_ptr() % 4 == 0 else None
        assert flat is not None
        return torch.as_strided(flat, (n, m), (int(ld.value), 1), storage_offset=int(offset))

    def pg_read_q(self, i: int, j: int, layer: int, stream=None) -> np.ndarray:
        """(cols, rank) array."""
        m = self.layer_shapes[layer][1]
        out = np.empty((self.rank, m), dtype=np.float32)
        _check(self._lib.pg_read_q(self._h, i, j, layer, out.ctypes.data, _stream_handle(stream)), "pg_read_q")
        return out.T.copy()

    def pg_write_q(self, i: int, j: int, layer: int, q: np.ndarray, stream=None) -> None:
        m = self.layer_shapes[layer][1]
        src = np.ascontiguousarray(np.asarray(q, dtype=np.float32).reshape(m, self.rank).T)
        _check(self._lib.pg_write_q(self._h, i, j, layer, src.ctypes.data, _stream_handle(stream)), "pg_write_q")

    # -- rounds -----------------------------------------------------------
    def pg_round(self, stream=None) -> None:
        _check(self._lib.pg_round(self._h, _stream_handle(stream)), "pg_round")

    def pg_stack_elems(self) -> int:
        n = ctypes.c_int64(0)
        _check(self._lib.pg_stack_elems(self._h, ctypes.byref(n)), "pg_stack_elems")
        return int(n.value)

    def pg_stack_offset(self, worker: int, layer: int):
        """(offset in floats, leading dimension) of a worker's matrix in a buffer shaped like the stack."""
        off, ld = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(self._lib.pg_stack_offset(self._h, worker, layer, ctypes.byref(off), ctypes.byref(ld)),
               "pg_stack_offset")
        return int(off.value), int(ld.value)

    def gradient_buffer(self):
        """A zeroed fp32 CUDA tensor of pg_stack_elems floats on the workspace's device."""
        import torch

        return torch.zeros(self.pg_stack_elems(), dtype=torch.float32, device=self._workspace.device)

    def gradient_view(self, grads, worker: int, layer: int):
        """(rows x cols) view of a worker's matrix inside a buffer made by gradient_buffer()."""
        import torch

        off, ld = self.pg_stack_offset(worker, layer)
        n, m = self.layer_shapes[layer]
        return torch.as_strided(grads, (n, m), (ld, 1), storage_offset=off)

    def pg_round_sgd(self, grads, eta: float, stream=None) -> None:
        """grads: fp32 CUDA tensor of pg_stack_elems floats laid out like the parameter stack."""
        import torch

        if not (isinstance(grads, torch.Tensor) and grads.is_cuda and grads.dtype == torch.float32
                and grads.is_contiguous() and grads.numel() >= self.pg_stack_elems()):
            raise ValueError("grads must be a contiguous fp32 CUDA tensor of at least pg_stack_elems floats")
        _check(self._lib.pg_round_sgd(self._h, ctypes.c_void_p(grads.data_ptr()), ctypes.c_float(eta),
                                      _stream_handle(stream)), "pg_round_sgd")

    def pg_set_half_step(self, on: bool = True) -> None:
        _check(self._lib.pg_set_half_step(self._h, 1 if on else 0), "pg_set_half_step")

    def pg_set_random_projection(self, mode: int) -> None:
        _check(self._lib.pg_set_random_projection(self._h, int(mode)), "pg_set_random_projection")

    def pg_rounds(self, n_rounds: int, stream=None) -> None:
        _check(self._lib.pg_rounds(self._h, int(n_rounds), _stream_handle(stream)), "pg_rounds")

    def pg_selftest_barrier_timeout(self, stream=None) -> int:
        return int(self._lib.pg_selftest_barrier_timeout(self._h, _stream_handle(stream)))

    def pg_selftest_bounds_check(self, stream=None) -> int:
        return int(self._lib.pg_selftest_bounds_check(self._h, _stream_handle(stream)))

    def pg_device_status(self, stream=None) -> int:
        return int(self._lib.pg_device_status(self._h, _stream_handle(stream)))

    def pg_get_schedule(self, round_index: int) -> Tuple[np.ndarray, np.ndarray]:
        cap = ctypes.c_int32(0)
        _check(self._lib.pg_max_edges(self._h, ctypes.byref(cap)), "pg_max_edges")
        edges = np.zeros((cap.value, 2), dtype=np.int32)
        w = np.zeros(cap.value, dtype=np.float32)
        n = ctypes.c_int32(0)
        _check(self._lib.pg_get_schedule(self._h, round_index, edges.ctypes.data, w.ctypes.data,
                                         ctypes.byref(n)), "pg_get_schedule")
        return edges[:n.value].copy(), w[:n.value].copy()

    def pg_get_round(self) -> int:
        r = ctypes.c_int64(0)
        _check(self._lib.pg_get_round(self._h, ctypes.byref(r)), "pg_get_round")
        return int(r.value)

    def pg_set_round(self, r: int, stream=None) -> None:
        _check(self._lib.pg_set_round(self._h, int(r), _stream_handle(stream)), "pg_set_round")

    def pg_comm_floats_round(self, round_index: int) -> Tuple[int, int]:
        """(floats all workers send in that round, floats uncompressed gossip would send)."""
        sent, dense = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(self._lib.pg_comm_floats_round(self._h, int(round_index), ctypes.byref(sent), ctypes.byref(dense)),
               "pg_comm_floats_round")
        return int(sent.value), int(dense.value)

    def pg_kernel_launches(self) -> int:
        r = ctypes.c_int64(0)
        _check(self._lib.pg_kernel_launches(self._h, ctypes.byref(r)), "pg_kernel_launches")
        return int(r.value)

    def pg_round_bytes(self) -> Tuple[float, float]:
        """(algorithmic bytes of X one steady-state round moves, share of the parameters on the pair sweep)."""
        b, f = ctypes.c_double(0.0), ctypes.c_double(0.0)
        _check(self._lib.pg_round_bytes(self._h, ctypes.byref(b), ctypes.byref(f)), "pg_round_bytes")
        return float(b.value), float(f.value)

    def pg_timing_enable(self, on: bool) -> None:
        _check(self._lib.pg_timing_enable(self._h, 1 if on else 0), "pg_timing_enable")

    def pg_timing_read(self):
        """{kernel kind: (total ms, launches, algorithmic bytes)} since the last read."""
        ms = np.zeros(len(KERNEL_KINDS), dtype=np.float64)
        cnt = np.zeros(len(KERNEL_KINDS), dtype=np.int64)
        nbytes = np.zeros(len(KERNEL_KINDS), dtype=np.float64)
        _check(self._lib.pg_timing_read(self._h, ms.ctypes.data, cnt.ctypes.data, nbytes.ctypes.data),
               "pg_timing_read")
        return {k: (float(ms[t]), int(cnt[t]), float(nbytes[t])) for t, k in enumerate(KERNEL_KINDS)}

    # -- conveniences built only from the calls above ---------------------
    def write_all(self, params: Sequence[Sequence[np.ndarray]], stream=None) -> None:
        for i, row in enumerate(params):
            for l, x in enumerate(row):
                self.pg_write_params(i, l, x, stream)

    def read_all(self, stream=None) -> List[List[np.ndarray]]:
        return [[self.pg_read_params(i, l, stream=stream) for l in range(len(self.layer_shapes))]
                for i in range(self.n_workers)]


def _host_ptr(x, shape):
    """Pointer to a dense fp32 host array (numpy or CPU torch tensor)."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.float32 or not x.flags["C_CONTIGUOUS"] or tuple(x.shape) != tuple(shape):
            raise ValueError("expected a C-contiguous float32 array of shape %r" % (tuple(shape),))
        return ctypes.c_void_p(x.ctypes.data), x
    import torch

    if isinstance(x, torch.Tensor):
        if x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous() or tuple(x.shape) != tuple(shape):
            raise ValueError("expected a contiguous float32 CPU tensor of shape %r" % (tuple(shape),))
        return ctypes.c_void_p(x.data_ptr()), x
    raise TypeError("expected a numpy array or a CPU torch tensor")
