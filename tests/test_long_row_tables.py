"""Host logic that cuts long rows of A + I into work items (one warp each): the items must tile every
long row exactly, respect the length limit, fall on community-segment boundaries wherever a segment
fits, and the tables that put the pieces back together must point at the right items.  No GPU."""
import os
import subprocess

import numpy as np
import pytest

from conftest import random_graph

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def harness(tmp_path_factory):
    exe = str(tmp_path_factory.mktemp("harness") / "long_row_tables")
    src = os.path.join(ROOT, "tests", "long_row_tables_harness.cpp")
    subprocess.run(["g++", "-O1", "-std=c++17", "-fopenmp", "-o", exe, src], check=True)
    return exe


def run(exe, row_ptr, col, comm, n_comm, limit):
    n = len(comm)
    text = f"{n} {n_comm} {limit}\n" + " ".join(map(str, row_ptr)) + "\n" + " ".join(map(str, col)) + "\n" + \
        " ".join(map(str, comm)) + "\n"
    out = subprocess.run([exe], input=text, capture_output=True, text=True, check=True).stdout.split("\n")
    it = iter(out)
    nnz = int(next(it))
    rp = np.array(next(it).split(), dtype=np.int64)
    cl = np.array(next(it).split(), dtype=np.int64)
    rc = np.array(next(it).split(), dtype=np.int64)
    assert len(cl) == nnz
    tabs = []
    for _ in range(3):
        k = int(next(it))
        tabs.append(np.array([next(it).split() for _ in range(k)], dtype=np.int64).reshape(k, 4))
    return rp, cl, rc, tabs


def hub_graph(rng, n, p, hubs):
    """A sparse random graph plus a few rows connected to a large share of all nodes."""
    _, _, A = random_graph(rng, n, p)
    for h in hubs:
        nb = rng.random(n) < 0.7
        A[h, nb] = 1
        A[nb, h] = 1
    np.fill_diagonal(A, 0)
    row_ptr = np.concatenate([[0], np.cumsum(A.sum(1))]).astype(np.int64)
    col = np.concatenate([np.nonzero(A[i])[0] for i in range(n)]).astype(np.int64)
    return row_ptr, col


@pytest.mark.parametrize("seed,n,n_comm,limit", [(0, 60, 3, 4), (1, 90, 5, 7), (2, 120, 2, 16), (3, 50, 1, 5),
                                                 (4, 80, 8, 1), (5, 70, 4, 1000)])
def test_items_tile_long_rows(harness, seed, n, n_comm, limit):
    rng = np.random.default_rng(seed)
    row_ptr, col = hub_graph(rng, n, 0.05, hubs=rng.choice(n, 4, replace=False))
    comm = rng.integers(0, n_comm, n)
    comm[:n_comm] = np.arange(n_comm)
    rp, cl, rc, (items, split, rows) = run(harness, row_ptr, col, comm, n_comm, limit)
    deg = np.diff(rp)
    long_rows = np.nonzero(deg > limit)[0]
    assert list(rows[:, 0]) == list(long_rows)                      # exactly the long rows, ascending
    if limit >= deg.max():
        assert len(items) == 0 and len(split) == 0
        return
    assert len(long_rows) > 0
    seen_split = set()
    at = 0
    for row, first, count, _ in rows:
        assert first == at and count >= 2
        at += count
        pos = rp[row]
        for k in range(first, first + count):
            r, b, e, sp = items[k]
            assert r == row and b == pos and e > b and e - b <= limit    # consecutive, non-empty, short enough
            pos = e
            cc = rc[cl[b:e]]
            left_is_cut = b == rp[row] or rc[cl[b - 1]] != cc[0]
            right_is_cut = e == rp[row + 1] or rc[cl[e]] != cc[-1]
            if sp < 0:
                assert left_is_cut and right_is_cut                       # whole segments only
            else:
                assert len(set(cc)) == 1                                  # a piece of one segment
                srow, scomm, sfirst, scount = split[sp]
                assert srow == row and scomm == cc[0] and sfirst <= k < sfirst + scount
                seen_split.add(sp)
        assert pos == rp[row + 1]                                         # the row is covered exactly
    assert at == len(items)
    assert seen_split == set(range(len(split)))
    for sp, (row, scomm, sfirst, scount) in enumerate(split):
        assert scount >= 2 and np.all(items[sfirst:sfirst + scount, 3] == sp)
        b, e = items[sfirst, 1], items[sfirst + scount - 1, 2]
        assert e - b > limit and np.all(rc[cl[b:e]] == scomm)             # the whole over-long segment ...
        assert (b == rp[row] or rc[cl[b - 1]] != scomm) and (e == rp[row + 1] or rc[cl[e]] != scomm)   # ... and all of it
