"""The allocation-free transposed product against the regular path (GPU).

Collected last on purpose (file name): a failure here cannot hide the result of
any other test in a run that stops at the first failure.

`pg_transposed_product_noalloc` serves callers that cannot allocate device
memory (allocator callbacks, fixed memory budgets, latency paths where
cudaMalloc's device-wide synchronisation is not acceptable): its partial sums
live in a fixed array inside the library.  Here its result is compared with
what the regular entry points produce for the same product.  In a two-worker
network whose second worker holds zeros, one round stores
Q' = X_0^T p_hat with p_hat = X_0 q_hat / ||X_0 q_hat||, and `pg_read_q`
returns it.  The same two products are formed with the new call: first
X_0 q_hat (as the transposed product of X_0^T), then X_0^T p_hat - two calls
in a row on the shared scratch - and the result must agree within the 1e-4
relative tolerance the parity tests use.
"""
import numpy as np
import pytest

from paper_2008_01425_b200 import workloads as wl

pytestmark = pytest.mark.gpu

REL_TOL = 1e-4


def _regular_path(x0, seed):
    """Q' and the initial q of a two-worker network through pg_create/pg_round/pg_read_q."""
    from paper_2008_01425_b200 import binding as pg

    n, m = x0.shape
    net = pg.PowerGossip(kind=pg.PG_MATCHING, n_workers=2, layer_shapes=[(n, m)], rank=1,
                         power_steps=1, seed=seed)
    net.pg_write_params(0, 0, x0)
    net.pg_write_params(1, 0, np.zeros_like(x0))
    q0 = net.pg_read_q(0, 1, 0)[:, 0].copy()
    net.pg_round()
    q_new = net.pg_read_q(0, 1, 0)[:, 0].copy()
    assert net.pg_device_status() == pg.PG_OK
    net.close()
    return q0, q_new


@pytest.mark.parametrize("shape", [(300, 132), (517, 131), (1, 9), (2600, 650)])
def test_two_calls_in_a_row_match_the_regular_path(shape):
    import torch

    from paper_2008_01425_b200 import binding as pg

    n, m = shape
    rng = np.random.default_rng(n * 1000 + m)
    x0 = rng.standard_normal((n, m)).astype(np.float32)
    q0, q_expected = _regular_path(x0, seed=31)

    dev = torch.device("cuda:0")
    X = torch.from_numpy(x0).to(dev)
    Xt = torch.from_numpy(np.ascontiguousarray(x0.T)).to(dev)
    q_hat = torch.from_numpy((q0.astype(np.float64) / np.linalg.norm(q0.astype(np.float64))).astype(np.float32)).to(dev)
    p = torch.empty(n, dtype=torch.float32, device=dev)
    z = torch.empty(m, dtype=torch.float32, device=dev)
    for attempt in range(2):          # the scratch keeps the previous call's contents: run it all twice
        p.fill_(float("nan"))
        z.fill_(float("nan"))
        pg.pg_transposed_product_noalloc(Xt, q_hat, p)          # p = (X_0^T)^T q_hat = X_0 q_hat
        p_hat = p / torch.linalg.vector_norm(p.double()).float()
        pg.pg_transposed_product_noalloc(X, p_hat, z)           # z = X_0^T p_hat
        torch.cuda.synchronize()
        got = z.cpu().numpy().astype(np.float64)
        err = np.linalg.norm(got - q_expected) / np.linalg.norm(q_expected)
        assert err <= REL_TOL, "attempt %d: relative error %.3e" % (attempt, err)
        # and each of the two products against the same product formed in double precision
        # from the very operands the call was given (numpy on the host)
        p_ref = x0.astype(np.float64) @ q_hat.cpu().numpy().astype(np.float64)
        z_ref = x0.astype(np.float64).T @ p_hat.cpu().numpy().astype(np.float64)
        for name, mine, ref in (("X q", p.cpu().numpy(), p_ref), ("X^T p", got, z_ref)):
            e64 = np.linalg.norm(mine.astype(np.float64) - ref) / np.linalg.norm(ref)
            assert e64 <= 1e-6, "attempt %d, %s: relative error %.3e against fp64" % (attempt, name, e64)


def test_strided_rows_and_rejection_of_oversized_problems():
    import torch

    from paper_2008_01425_b200 import binding as pg

    dev = torch.device("cuda:0")
    rng = np.random.default_rng(5)
    big = torch.from_numpy(rng.standard_normal((70, 40)).astype(np.float32)).to(dev)
    view = big[:, :33]                                          # leading dimension 40, 33 columns
    p = torch.from_numpy(rng.standard_normal(70).astype(np.float32)).to(dev)
    z = torch.empty(33, dtype=torch.float32, device=dev)
    pg.pg_transposed_product_noalloc(view, p, z)
    torch.cuda.synchronize()
    ref = view.double().T @ p.double()
    assert float(torch.linalg.vector_norm(z.double() - ref) / torch.linalg.vector_norm(ref)) <= 1e-6
    # ceil(rows/256) * cols beyond the fixed scratch: refused, nothing launched
    rows, cols = 256 * 9, pg.PG_NOALLOC_MAX_PARTIALS // 8
    with pytest.raises(pg.PowerGossipError) as e:
        pg.pg_transposed_product_noalloc(big, p, z, rows=rows, cols=cols, ld=cols)
    assert e.value.status == pg.PG_ERR_TOO_LARGE
    with pytest.raises(pg.PowerGossipError) as e:
        pg.pg_transposed_product_noalloc(big, p, z, rows=0, cols=4, ld=4)
    assert e.value.status == pg.PG_ERR_INVALID
    # more row tiles than one launch can hold, although their partial sums would fit the scratch;
    # and a column count whose rounding up would overflow: both refused on the host, z untouched
    z.fill_(7.0)
    for rows, cols in ((256 * 65536, 8), (1, 2 ** 31 - 2)):
        with pytest.raises(pg.PowerGossipError) as e:
            pg.pg_transposed_product_noalloc(big, p, z, rows=rows, cols=cols, ld=cols)
        assert e.value.status == pg.PG_ERR_TOO_LARGE, (rows, cols)
    torch.cuda.synchronize()
    assert bool((z == 7.0).all())
