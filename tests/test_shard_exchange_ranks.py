"""The exchange that the multi-GPU plan describes (Section 2: one agent per community group; Appendix A,
Eq. 4: first- and second-order messages; Section 3.1: the agent that sums the W gradients), carried out by
gloo ranks on the CPU: every rank keeps only its own rows, receives the first-order rows its plan lists
from their owners, and must then be able to form its rows of A~ X; a second exchange of the result gives
its rows of A~ A~ X (what the second-order message carries, computed by the rows' owners instead of
being sent two hops); the per-rank P^T R summed by all-reduce is the full gradient.  No GPU."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _exchange(rank, world, first, row_begin, M):
    """Rows of M (all ranks hold an array of the full shape, valid on their own rows only) that `rank`
    needs from the others arrive in place; everything else stays NaN."""
    ops, bufs = [], {}
    for other in range(world):
        if other == rank:
            continue
        send_rows = first[(other, rank)]          # what `other` receives from this rank
        recv_rows = first[(rank, other)]
        if len(send_rows):
            ops.append(dist.P2POp(dist.isend, torch.from_numpy(np.ascontiguousarray(M[send_rows])), other))
        if len(recv_rows):
            bufs[other] = torch.empty((len(recv_rows), M.shape[1]), dtype=torch.float64)
            ops.append(dist.P2POp(dist.irecv, bufs[other], other))
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    for other, buf in bufs.items():
        assert ((first[(rank, other)] >= row_begin[other]) & (first[(rank, other)] < row_begin[other + 1])).all()
        M[first[(rank, other)]] = buf.numpy()


def _worker(rank, world, port, exe, seed, n, n_comm, p, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from conftest import random_graph
    from oracle import gcn_admm_oracle as orc
    from test_shard_plan import run
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(seed)              # every rank builds the same problem, then forgets what it does not own
    row_ptr, col, _ = random_graph(rng, n, p)
    comm = rng.integers(0, n_comm, n)
    comm[:n_comm] = np.arange(n_comm)
    X = rng.standard_normal((n, 3))
    R = rng.standard_normal((n, 2))
    _, row_begin, first, _ = run(exe, row_ptr, col, comm, n_comm, world)
    ix = orc.community_index(n, row_ptr, col, comm, n_comm)
    perm = ix["perm"]
    At = orc.normalized_adjacency(n, row_ptr, col)[perm][:, perm].tocsr()
    Xp, Rp = X[perm], R[perm]
    own = np.arange(row_begin[rank], row_begin[rank + 1])

    def own_rows_of_product(M):
        """A~[own] M from the rows this rank holds; a NaN in the result means a row was missing."""
        res = np.full((len(own), M.shape[1]), np.nan)
        for k, i in enumerate(own):
            cols = At.indices[At.indptr[i]:At.indptr[i + 1]]
            vals = At.data[At.indptr[i]:At.indptr[i + 1]]
            res[k] = vals @ M[cols]
        return res

    mine = np.full_like(Xp, np.nan)
    mine[own] = Xp[own]
    _exchange(rank, world, first, row_begin, mine)
    P_own = own_rows_of_product(mine)
    assert np.isfinite(P_own).all()
    full_P = At @ Xp
    err1 = float(np.abs(P_own - full_P[own]).max())
    # second hop: owners exchange their rows of P, no second-order row travels
    Pm = np.full_like(Xp, np.nan)
    Pm[own] = P_own
    _exchange(rank, world, first, row_begin, Pm)
    Q_own = own_rows_of_product(Pm)
    assert np.isfinite(Q_own).all()
    err2 = float(np.abs(Q_own - (At @ full_P)[own]).max())
    # the gradient of a W block: per-rank P^T R, summed over the ranks
    g = torch.from_numpy(P_own.T @ Rp[own])
    dist.all_reduce(g)
    err3 = float(np.abs(g.numpy() - full_P.T @ Rp).max())
    received = sum(len(first[(rank, s)]) for s in range(world))
    out[rank] = (err1, err2, err3, len(own), received)
    dist.barrier()
    dist.destroy_process_group()


def _harness(tmp_path):
    exe = str(tmp_path / "shard_plan")
    subprocess.run(["g++", "-O1", "-std=c++17", "-fopenmp", "-o", exe, os.path.join(ROOT, "tests", "shard_plan_harness.cpp")],
                   check=True)
    return exe


def _run(tmp_path, world, seed, n, n_comm, p):
    exe = _harness(tmp_path)
    port = 31000 + (os.getpid() * 7 + world) % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, exe, seed, n, n_comm, p, out), nprocs=world, join=True)
        return dict(out)


def test_two_ranks_exchange_first_order_rows(tmp_path):
    out = _run(tmp_path, 2, seed=5, n=60, n_comm=6, p=0.06)
    assert sum(v[3] for v in out.values()) == 60            # the ranks' own rows cover the graph
    assert any(v[4] > 0 for v in out.values())              # and something did travel
    for rank, (e1, e2, e3, _, _) in out.items():
        assert e1 < 1e-13 and e2 < 1e-13 and e3 < 1e-12, (rank, e1, e2, e3)


def test_three_ranks_exchange_first_order_rows(tmp_path):
    out = _run(tmp_path, 3, seed=11, n=90, n_comm=9, p=0.04)
    assert sum(v[3] for v in out.values()) == 90
    for rank, (e1, e2, e3, _, _) in out.items():
        assert e1 < 1e-13 and e2 < 1e-13 and e3 < 1e-12, (rank, e1, e2, e3)
