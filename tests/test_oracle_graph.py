"""Pins of the oracle's graph side: the normalised adjacency and the community index sets.
None of these checks re-uses the oracle's own formulas: they use dense brute force, closed
forms for special graphs and a hand-made example."""
import os

import numpy as np
import pytest

from conftest import dense_to_csr, random_graph
from oracle import gcn_admm_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def dense_At(A):
    n = A.shape[0]
    d = A.sum(axis=1) + 1.0
    B = A + np.eye(n)
    out = np.zeros((n, n))
    for i in range(n):
        for j in range(n):
            out[i, j] = B[i, j] / np.sqrt(d[i] * d[j])
    return out


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_adjacency_matches_dense_brute_force(seed):
    rng = np.random.default_rng(seed)
    row_ptr, col_idx, A = random_graph(rng, 17, 0.25)
    At = orc.normalized_adjacency(17, row_ptr, col_idx).toarray()
    np.testing.assert_allclose(At, dense_At(A), rtol=0, atol=1e-15)
    assert np.array_equal(At, At.T) or np.allclose(At, At.T, atol=1e-16)
    assert (At >= 0).all()
    sd = np.sqrt(A.sum(axis=1) + 1.0)
    np.testing.assert_allclose(At @ sd, sd, rtol=1e-14)       # (A+I) 1 = d


def test_adjacency_special_graphs():
    n = 7
    K = np.ones((n, n)) - np.eye(n)
    At = orc.normalized_adjacency(n, *dense_to_csr(K)).toarray()
    np.testing.assert_allclose(At, np.full((n, n), 1.0 / n), atol=1e-15)
    ring = np.zeros((n, n))
    for i in range(n):
        ring[i, (i + 1) % n] = ring[(i + 1) % n, i] = 1
    At = orc.normalized_adjacency(n, *dense_to_csr(ring)).toarray()
    np.testing.assert_allclose(At, (ring + np.eye(n)) / 3.0, atol=1e-15)
    At = orc.normalized_adjacency(n, *dense_to_csr(np.zeros((n, n)))).toarray()
    np.testing.assert_allclose(At, np.eye(n), atol=0)


def test_adjacency_ignores_input_self_loops():
    rng = np.random.default_rng(3)
    _, _, A = random_graph(rng, 9, 0.3)
    B = A + np.diag(rng.integers(0, 2, 9))
    a = orc.normalized_adjacency(9, *dense_to_csr(A)).toarray()
    b = orc.normalized_adjacency(9, *dense_to_csr(B)).toarray()
    np.testing.assert_array_equal(a, b)


def brute_index(A, community, M):
    """Index sets straight from the definitions, O(N^2) on a dense matrix, original ids."""
    n = A.shape[0]
    nbr, h1, h2 = [], [], []
    for m in range(M):
        own = [i for i in range(n) if community[i] == m]
        first = sorted({j for i in own for j in range(n) if A[i, j] and community[j] != m})
        second = sorted({k for j in first for k in range(n)
                         if A[j, k] and community[k] != m and k not in first})
        nbr.append(sorted({int(community[j]) for j in first}))
        h1.append(first)
        h2.append(second)
    return nbr, h1, h2


@pytest.mark.parametrize("seed,M", [(0, 3), (1, 4), (2, 1), (3, 5)])
def test_index_matches_brute_force(seed, M):
    rng = np.random.default_rng(seed)
    n = 30
    row_ptr, col_idx, A = random_graph(rng, n, 0.12)
    community = rng.integers(0, M, size=n)
    community[:M] = np.arange(M)
    ix = orc.community_index(n, row_ptr, col_idx, community, M)
    perm, inv = ix["perm"], ix["inv"]
    # ordering: by (community, original id)
    expect = sorted(range(n), key=lambda i: (community[i], i))
    assert perm.tolist() == expect
    assert inv[perm].tolist() == list(range(n))
    assert ix["comm_ptr"].tolist() == [int((community < m).sum()) for m in range(M + 1)]
    nbr, h1, h2 = brute_index(A, community, M)
    for m in range(M):
        assert ix["nbr"][m].tolist() == nbr[m]
        assert sorted(perm[ix["halo1"][m]].tolist()) == h1[m]
        assert sorted(perm[ix["halo2"][m]].tolist()) == h2[m]
        assert np.all(np.diff(ix["halo1"][m]) > 0) and np.all(np.diff(ix["halo2"][m]) > 0)
    if M == 1:
        assert all(len(x) == 0 for x in ix["halo1"] + ix["halo2"] + ix["nbr"])
    # every cross edge (u, v) has v in halo1(comm(u))
    for u in range(n):
        for v in range(n):
            if A[u, v] and community[u] != community[v]:
                assert inv[v] in ix["halo1"][community[u]]
    # permuted CSR of A+I, and its segments
    B = (A + np.eye(n))[np.ix_(perm, perm)]
    comm_new = community[perm]
    for i in range(n):
        lo, hi = ix["csr_row_ptr"][i], ix["csr_row_ptr"][i + 1]
        assert ix["csr_col"][lo:hi].tolist() == np.flatnonzero(B[i]).tolist()
        s0, s1 = ix["seg_row_ptr"][i], ix["seg_row_ptr"][i + 1]
        assert ix["seg_begin"][s0] == lo and ix["seg_begin"][s1] == hi
        covered = []
        for s in range(s0, s1):
            cols = ix["csr_col"][ix["seg_begin"][s]:ix["seg_begin"][s + 1]]
            assert len(cols) > 0 and (comm_new[cols] == ix["seg_comm"][s]).all()
            covered += cols.tolist()
        assert covered == ix["csr_col"][lo:hi].tolist()
        assert np.all(np.diff(ix["seg_comm"][s0:s1]) > 0)


def test_worked_example_three_communities():
    spec = {}
    for line in open(os.path.join(GOLDEN, "three_communities.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *rest = line.split()
        spec[key] = rest
    names = [t.split(":")[0] for t in spec["nodes"]]
    community = np.array([int(t.split(":")[1]) - 1 for t in spec["nodes"]])
    n = len(names)
    A = np.zeros((n, n))
    for e in spec["edges"]:
        a, b = e.split("-")
        A[names.index(a), names.index(b)] = A[names.index(b), names.index(a)] = 1
    ix = orc.community_index(n, *dense_to_csr(A), community, 3)
    for t in spec["N"]:
        m, lst = t.split(":")
        assert (ix["nbr"][int(m) - 1] + 1).tolist() == [int(x) for x in lst.split(",")]
    for key in ("halo1", "halo2"):
        for t in spec[key]:
            m, lst = t.split(":")
            got = sorted(names[ix["perm"][j]] for j in ix[key][int(m) - 1])
            assert got == sorted(lst.split(","))
    assert (ix["nbr"][0] + 1).tolist() == [3]          # the sentence of Section 2
