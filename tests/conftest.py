import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def random_graph(rng, n, p):
    """Symmetric simple graph as (row_ptr int64, col_idx int32) plus its dense 0/1 matrix."""
    A = np.triu(rng.random((n, n)) < p, k=1)
    A = (A | A.T).astype(np.float64)
    return dense_to_csr(A) + (A,)


def dense_to_csr(A):
    n = A.shape[0]
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    cols = []
    for i in range(n):
        c = np.flatnonzero(A[i])
        cols.append(c)
        row_ptr[i + 1] = row_ptr[i] + len(c)
    col_idx = np.concatenate(cols).astype(np.int32) if n else np.zeros(0, dtype=np.int32)
    return row_ptr, col_idx


def tiny_problem(seed, n=24, widths=(5, 6, 4, 3), n_comm=3, p=0.2, n_train=None):
    """A small random instance: graph, features, labels, mask, communities, weights."""
    rng = np.random.default_rng(seed)
    row_ptr, col_idx, A = random_graph(rng, n, p)
    X = rng.standard_normal((n, widths[0]))
    y = rng.integers(0, widths[-1], size=n)
    mask = np.zeros(n, dtype=np.uint8)
    mask[rng.choice(n, size=n_train or max(n // 3, 1), replace=False)] = 1
    community = rng.integers(0, n_comm, size=n)
    community[:n_comm] = np.arange(n_comm)          # no empty community
    W = [rng.standard_normal((widths[l], widths[l + 1])) * 0.5 for l in range(len(widths) - 1)]
    return dict(n=n, row_ptr=row_ptr, col_idx=col_idx, A=A, X=X, y=y, mask=mask,
                community=community, n_comm=n_comm, widths=list(widths), W=W)


@pytest.fixture
def rng():
    return np.random.default_rng(12345)
