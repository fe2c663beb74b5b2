"""Host-side index build (Section 2: V_m, N_m and the block split of A~; Appendix A: the rows a community
depends on): the library's tables against the oracle's, bit for bit, and the input checks, without a GPU.
The library's code runs in a small host program (the harness shared with the shard-plan test)."""
import os
import subprocess

import numpy as np
import pytest

from conftest import random_graph
from oracle import gcn_admm_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def harness(tmp_path_factory):
    exe = str(tmp_path_factory.mktemp("harness") / "graph_index")
    src = os.path.join(ROOT, "tests", "shard_plan_harness.cpp")
    subprocess.run(["g++", "-O1", "-std=c++17", "-fopenmp", "-o", exe, src], check=True)
    return exe


def run(exe, row_ptr, col, comm, n_comm, threads=3):
    n = len(comm)
    text = f"{n} {n_comm} 1\n" + " ".join(map(str, row_ptr)) + "\n" + " ".join(map(str, col)) + "\n" + \
        " ".join(map(str, comm)) + "\n"
    env = dict(os.environ, OMP_NUM_THREADS=str(threads))
    res = subprocess.run([exe, "index"], input=text, capture_output=True, text=True, env=env)
    if res.returncode != 0:
        return res.returncode, res.stderr.strip()
    lines = res.stdout.split("\n")
    assert lines[0] == "ok"
    names = ["perm", "inv", "comm_ptr", "row_comm", "row_ptr", "col", "col_comm", "seg_row_ptr", "seg_comm", "seg_begin"]
    out = {k: np.array(lines[1 + i].split()[1:], dtype=np.int64) for i, k in enumerate(names)}
    out["dinv"] = np.array(lines[1 + len(names)].split(), dtype=np.float64)
    return 0, out


def with_self_loops(rng, row_ptr, col, share):
    """The same graph with a diagonal entry added to some rows (the library drops them and adds the identity)."""
    n = len(row_ptr) - 1
    rows = []
    for i in range(n):
        r = list(col[row_ptr[i]:row_ptr[i + 1]])
        if rng.random() < share:
            r = sorted(r + [i])
        rows.append(r)
    rp = np.concatenate([[0], np.cumsum([len(r) for r in rows])]).astype(np.int64)
    return rp, np.array([c for r in rows for c in r], dtype=np.int32)


@pytest.mark.parametrize("seed,n,n_comm,p,loops", [(0, 60, 5, 0.1, 0.0), (1, 90, 9, 0.05, 0.3), (2, 40, 40, 0.2, 1.0),
                                                   (3, 70, 3, 0.0, 0.5), (4, 300, 64, 0.04, 0.1), (5, 120, 1, 0.1, 0.2),
                                                   (6, 200, 150, 0.3, 0.0)])
def test_tables_equal_the_oracles(harness, seed, n, n_comm, p, loops):
    rng = np.random.default_rng(seed)
    row_ptr, col, _ = random_graph(rng, n, p)
    comm = rng.integers(0, n_comm, n)
    comm[:n_comm] = rng.permutation(n_comm)
    ix = orc.community_index(n, row_ptr, col, comm, n_comm)
    rp2, col2 = with_self_loops(rng, row_ptr, col, loops)
    for threads in (1, 3):
        rc, got = run(harness, rp2, col2, comm, n_comm, threads)
        assert rc == 0, got
        for name, key in (("perm", "perm"), ("inv", "inv"), ("comm_ptr", "comm_ptr"), ("row_ptr", "csr_row_ptr"),
                          ("col", "csr_col"), ("seg_row_ptr", "seg_row_ptr"), ("seg_comm", "seg_comm"),
                          ("seg_begin", "seg_begin")):
            assert np.array_equal(got[name], ix[key]), name
        assert np.array_equal(got["row_comm"], comm[ix["perm"]])
        assert np.array_equal(got["col_comm"], got["row_comm"][got["col"]])
        deg = np.diff(row_ptr)                               # the graph without the added diagonal entries
        np.testing.assert_allclose(got["dinv"], 1.0 / np.sqrt(deg[ix["perm"]] + 1.0), rtol=1e-7)


def test_asymmetric_inputs_are_refused(harness):
    """The symmetry check compares fingerprints of the entry sets above and below the diagonal: one missing
    mirror, one extra entry, and a mirror moved to another place (equal counts on both sides) must all fail."""
    rng = np.random.default_rng(11)
    n = 50
    row_ptr, col, A = random_graph(rng, n, 0.15)
    comm = np.arange(n) % 4

    def csr(M):
        rp = np.concatenate([[0], np.cumsum((M > 0).sum(axis=1))]).astype(np.int64)
        return rp, np.nonzero(M > 0)[1].astype(np.int32)

    assert run(harness, *csr(A), comm, 4)[0] == 0
    i, j = np.argwhere(np.triu(A, 1) > 0)[3]
    B = A.copy(); B[j, i] = 0                                 # a mirror missing
    assert run(harness, *csr(B), comm, 4) == (3, "adjacency is not symmetric")
    a, b = np.argwhere((np.triu(np.ones_like(A), 1) > 0) & (A == 0))[5]
    B = A.copy(); B[a, b] = 1                                 # an entry without a mirror
    assert run(harness, *csr(B), comm, 4) == (3, "adjacency is not symmetric")
    B = A.copy(); B[j, i] = 0
    c, d = np.argwhere((np.tril(np.ones_like(A), -1) > 0) & (A == 0))[7]
    B[c, d] = 1                                               # as many entries below as above, one in the wrong place
    assert (np.triu(B, 1) > 0).sum() == (np.tril(B, -1) > 0).sum()
    assert run(harness, *csr(B), comm, 4) == (3, "adjacency is not symmetric")


def test_other_bad_inputs_are_refused(harness):
    rng = np.random.default_rng(12)
    n = 30
    row_ptr, col, _ = random_graph(rng, n, 0.2)
    comm = np.arange(n) % 3
    bad = col.copy(); bad[0] = n
    assert run(harness, row_ptr, bad, comm, 3) == (3, "column index out of range")
    i = int(np.argmax(np.diff(row_ptr) >= 2))
    swapped = col.copy(); p = row_ptr[i]; swapped[p], swapped[p + 1] = swapped[p + 1], swapped[p]
    assert run(harness, row_ptr, swapped, comm, 3) == (3, "columns of a row are not strictly ascending")
    assert run(harness, row_ptr, col, comm + 1, 3)[0] == 3      # community id out of range
    assert run(harness, row_ptr, col, np.zeros(n, int), 2) == (3, "empty community")
