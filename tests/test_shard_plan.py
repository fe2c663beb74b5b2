"""Host-side plan for spreading communities over several GPUs (Section 2: a community per agent; Appendix A,
Eq. 4: first- and second-order messages): contiguous community ranges per rank and, for every ordered pair
of ranks, the first-order and second-order rows the receiver depends on.  Checked against lists derived
from the oracle's index sets and, on tiny graphs, against brute force on the dense adjacency.  No GPU."""
import os
import subprocess

import numpy as np
import pytest

from conftest import random_graph
from oracle import gcn_admm_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def harness(tmp_path_factory):
    exe = str(tmp_path_factory.mktemp("harness") / "shard_plan")
    src = os.path.join(ROOT, "tests", "shard_plan_harness.cpp")
    subprocess.run(["g++", "-O1", "-std=c++17", "-fopenmp", "-o", exe, src], check=True)
    return exe


def run(exe, row_ptr, col, comm, n_comm, n_ranks):
    n = len(comm)
    text = f"{n} {n_comm} {n_ranks}\n" + " ".join(map(str, row_ptr)) + "\n" + " ".join(map(str, col)) + "\n" + \
        " ".join(map(str, comm)) + "\n"
    out = subprocess.run([exe], input=text, capture_output=True, text=True, check=True).stdout.split("\n")
    if out[0] != "ok":
        return None
    comm_begin = np.array(out[1].split(), dtype=np.int64)
    row_begin = np.array(out[2].split(), dtype=np.int64)
    lists = [np.array(line.split()[1:], dtype=np.int64) for line in out[3:3 + 2 * n_ranks * n_ranks]]
    first = {(r, s): lists[r * n_ranks + s] for r in range(n_ranks) for s in range(n_ranks)}
    second = {(r, s): lists[n_ranks * n_ranks + r * n_ranks + s] for r in range(n_ranks) for s in range(n_ranks)}
    return comm_begin, row_begin, first, second


@pytest.mark.parametrize("seed,n,n_comm,n_ranks,p", [(0, 40, 6, 2, 0.08), (1, 60, 9, 4, 0.05), (2, 50, 5, 5, 0.1),
                                                     (3, 30, 4, 1, 0.2), (4, 80, 12, 3, 0.03)])
def test_plan_against_oracle_index_sets_and_brute_force(harness, seed, n, n_comm, n_ranks, p):
    rng = np.random.default_rng(seed)
    row_ptr, col, A = random_graph(rng, n, p)
    comm = rng.integers(0, n_comm, n)
    comm[:n_comm] = np.arange(n_comm)
    comm_begin, row_begin, first, second = run(harness, row_ptr, col, comm, n_comm, n_ranks)
    ix = orc.community_index(n, row_ptr, col, comm, n_comm)
    # ranks own contiguous, non-empty community ranges that cover everything
    assert comm_begin[0] == 0 and comm_begin[-1] == n_comm and (np.diff(comm_begin) >= 1).all()
    assert np.array_equal(row_begin, ix["comm_ptr"][comm_begin])
    # balance: no rank holds more than its share of stored entries plus one community's worth
    nnz_of_comm = np.diff(ix["csr_row_ptr"][ix["comm_ptr"]])
    share = ix["csr_row_ptr"][-1] / n_ranks
    for r in range(n_ranks):
        assert nnz_of_comm[comm_begin[r]:comm_begin[r + 1]].sum() <= share + 2 * nnz_of_comm.max()
    rank_of = np.repeat(np.arange(n_ranks), np.diff(row_begin))
    # dense adjacency in new ids (brute force side)
    perm = ix["perm"]
    B = (A[np.ix_(perm, perm)] > 0)
    for r in range(n_ranks):
        own = np.arange(row_begin[r], row_begin[r + 1])
        # first-order rows from the oracle's per-community halo lists: union over r's communities, minus own rows
        h1 = np.unique(np.concatenate([ix["halo1"][m] for m in range(comm_begin[r], comm_begin[r + 1])] + [np.zeros(0, np.int64)]))
        h1 = h1[(h1 < row_begin[r]) | (h1 >= row_begin[r + 1])]
        brute1 = np.flatnonzero(B[own].any(axis=0))
        brute1 = np.setdiff1d(brute1, own)
        assert np.array_equal(h1, brute1)
        outside = np.setdiff1d(np.arange(n), np.union1d(own, brute1))
        brute2 = outside[B[np.ix_(brute1, outside)].any(axis=0)] if len(brute1) else np.zeros(0, np.int64)
        for s in range(n_ranks):
            assert np.array_equal(first[(r, s)], h1[rank_of[h1] == s]), (r, s)
            assert np.array_equal(second[(r, s)], brute2[rank_of[brute2] == s]), (r, s)
        assert len(first[(r, r)]) == 0 and len(second[(r, r)]) == 0
    # a send list is the receive list seen from the other side: s must own what r receives from it
    for (r, s), rows in first.items():
        assert ((rows >= row_begin[s]) & (rows < row_begin[s + 1])).all()
    # what the exchange is for: with the first-order rows in hand a rank can form its rows of A~ X
    At = orc.normalized_adjacency(n, row_ptr, col)[perm][:, perm].toarray()
    X = rng.standard_normal((n, 3))
    for r in range(n_ranks):
        own = np.arange(row_begin[r], row_begin[r + 1])
        have = np.union1d(own, np.concatenate([first[(r, s)] for s in range(n_ranks)] + [np.zeros(0, np.int64)])).astype(int)
        Xl = np.zeros_like(X)
        Xl[have] = X[have]
        np.testing.assert_allclose(At[own] @ Xl, At[own] @ X, atol=1e-14)


def test_more_ranks_than_communities_is_refused(harness):
    rng = np.random.default_rng(9)
    row_ptr, col, _ = random_graph(rng, 20, 0.2)
    comm = np.arange(20) % 3
    assert run(harness, row_ptr, col, comm, 3, 4) is None
    assert run(harness, row_ptr, col, comm, 3, 3) is not None
