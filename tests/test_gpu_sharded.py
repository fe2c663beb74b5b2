"""The propagation carried out rank by rank from local tables (each rank's own rows plus copies of its
first-order rows, columns renumbered to the local matrix) against the oracle's A~ X and against the unsharded
kernel: what every GPU of a sharded run would compute between two exchanges, run here one rank after the
other on one device (Section 2: every agent forms its rows from its own and its neighbours' first-order rows)."""
import numpy as np
import pytest

from paper_2112_09335_b200 import inputs
from parity_utils import make_pair, relerr

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[("cfg1", 1, 1.0), ("cfg3@0.012", 3, 0.012), ("cfg4@0.001", 4, 0.001)],
                ids=lambda c: c[0])
def case(request):
    _, cfg, scale = request.param
    wl = inputs.make_workload(cfg) if scale == 1.0 else inputs.make_workload(cfg, scale=scale)
    g, o = make_pair(wl)
    yield wl, g, o
    g.destroy()


@pytest.mark.parametrize("n_ranks", [1, 2, 3, 8])
@pytest.mark.parametrize("width", [3, 47, 256])
def test_rank_by_rank_propagation(case, n_ranks, width):
    wl, g, o = case
    n_ranks = min(n_ranks, wl.n_comm)
    rng = np.random.default_rng(width + n_ranks)
    x = rng.standard_normal((wl.n, width)).astype(np.float32)
    got, staged = g.propagate_sharded(n_ranks, x)
    want = o.At @ x.astype(np.float64)
    assert relerr(got, want) < 2e-7
    scale = np.abs(o.At) @ np.abs(x.astype(np.float64)) + 1e-30
    assert np.max(np.abs(got - want) / scale) < 1e-6          # every row
    whole = g.propagate(x)
    # same entry order in every row: the same bits as the unsharded kernel wherever that one walks a row whole
    rows = g.index("csr_row_ptr")
    short = np.diff(rows)[g.index("inv_perm")] <= 256        # default long_row; per original node
    assert np.array_equal(got[short], whole[short])
    assert np.max(np.abs(got - whole) / scale) < 1e-6
    # volume: one rank copies nothing, several copy exactly the plan's first-order rows
    planned = sum(len(g.shard_plan(n_ranks, 1, r, s)) for r in range(n_ranks) for s in range(n_ranks))
    assert staged == planned and (n_ranks > 1 or staged == 0)


def test_more_ranks_than_communities_is_refused(case):
    wl, g, _ = case
    x = np.zeros((wl.n, 4), dtype=np.float32)
    with pytest.raises(Exception):
        g.propagate_sharded(wl.n_comm + 1, x)
    g.propagate_sharded(wl.n_comm, x)          # the handle is still usable


def test_rank_sums_of_the_weight_gradient(case):
    """Section 3.1: the W agent adds up what the community agents send.  P^T R over each rank's row range by the
    library's transposed product, summed over the ranks (the all-reduce), against fp64 and the unsharded product."""
    import torch
    wl, g, _ = case
    n_ranks = min(4, wl.n_comm)
    ranges = g.shard_plan(n_ranks, 0)
    row_begin = ranges[n_ranks + 1:]
    rng = np.random.default_rng(3)
    ka, nb = 37, 24
    p = rng.standard_normal((wl.n, ka)).astype(np.float32)
    r = rng.standard_normal((wl.n, nb)).astype(np.float32)
    tp, tr = torch.from_numpy(p).cuda(), torch.from_numpy(r).cuda()
    whole = torch.empty((ka, nb), device="cuda")
    g.dense_product_tn(tp.data_ptr(), tr.data_ptr(), whole.data_ptr(), wl.n, ka, nb)
    total = np.zeros((ka, nb))
    for k in range(n_ranks):
        lo, hi = int(row_begin[k]), int(row_begin[k + 1])
        part = torch.empty((ka, nb), device="cuda")
        g.dense_product_tn(tp[lo:hi].data_ptr(), tr[lo:hi].data_ptr(), part.data_ptr(), hi - lo, ka, nb)
        total += part.cpu().numpy().astype(np.float64)
    want = p.astype(np.float64).T @ r.astype(np.float64)
    scale = np.abs(p).astype(np.float64).T @ np.abs(r).astype(np.float64)
    assert np.max(np.abs(total - want) / scale) < 2e-6
    assert np.max(np.abs(total - whole.cpu().numpy()) / scale) < 2e-6
