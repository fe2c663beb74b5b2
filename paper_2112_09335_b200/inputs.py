"""Seeded synthetic inputs for the community-based ADMM GCN trainer.

Nothing in this module belongs to the method: it only draws graphs, features,
labels, masks, initial weights and a community assignment.  Both the CUDA
library's tests/benchmark and the CPU oracle's tests are fed from here, so the
two implementations see the same numbers without sharing any arithmetic.

Six workload shapes are provided (``CONFIGS``; the sixth follows the sizes of the paper's own experiment).  They are synthetic stand-ins
with the node counts, degree distributions, feature shapes and label structure
of small citation graphs, a medium citation graph and two large co-purchase /
product graphs; no item of any public dataset is reproduced.  ``scale`` shrinks
the node and edge counts of a shape (same recipe) for cases a slow CPU program
can finish in seconds.

Recipe, per config index c (seed = BASE_SEED + c, numpy PCG64 streams):

* c = 0: stochastic block model, 4 equal blocks, edge probability 0.03 inside a
  block and 0.002 across; features Bernoulli(0.02) in {0,1}; every block picks a
  primary class out of 7, a node keeps it with probability 0.8 and otherwise
  draws uniformly; 140 training nodes without replacement.
* c >= 1: degree-corrected block model.  Node weights w_i = u^(-1/alpha) (a
  Pareto tail, alpha = degree exponent - 1) clipped so that no expected degree
  exceeds sqrt(N * mean degree); ``draw_factor * |E|`` edges are drawn with the
  first endpoint ~ w and the second ~ w inside the first endpoint's block with
  probability 0.85, else ~ w over all nodes; self loops and duplicates are
  dropped.  Node ids are then shuffled so that blocks are not contiguous.
* ADMM communities: the planted blocks when M equals their number, otherwise
  nodes sorted by (block, breadth-first position from the highest-degree node)
  and cut into M contiguous, equally sized chunks (node of rank r goes to chunk floor(r M / N)).
* Initial weights: Glorot-uniform.
"""

from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import scipy.sparse as sp
from scipy.sparse.csgraph import breadth_first_order

BASE_SEED = 211209335


@dataclass
class Workload:
    name: str
    n: int
    row_ptr: np.ndarray      # int64 [n+1], CSR of A (symmetric, sorted, no self loops)
    col_idx: np.ndarray      # int32 [nnz]
    X: np.ndarray            # float32 [n, C_0]
    y: np.ndarray            # int32 [n]
    train_mask: np.ndarray   # uint8 [n]
    widths: list             # C_0 .. C_L
    n_comm: int
    community: np.ndarray    # int32 [n], values 0..n_comm-1
    w_init: list             # L float32 arrays, C_{l-1} x C_l
    n_iters: int
    block: np.ndarray = field(default=None)  # planted block per node (int32)
    nu: float = 1e-3
    rho: float = 1e-3

    @property
    def n_edges(self) -> int:
        return int(self.col_idx.shape[0] // 2)


CONFIGS = [
    dict(name="tiny-sbm", n=1000, kind="sbm", blocks=4, p_in=0.03, p_out=0.002,
         feat="bernoulli", feat_p=0.02, c0=128, classes=7, label="noisy-block",
         train=140, widths=[128, 16, 7], n_comm=4, n_iters=10),
    dict(name="citation-small", n=2708, kind="dcsbm", blocks=7, edges=5300, alpha=1.5,
         draw_factor=1.065, feat="bow", feat_p=0.013, c0=1433, classes=7, label="block",
         train=140, widths=[1433, 16, 7], n_comm=8, n_iters=100),
    dict(name="citation-medium", n=19717, kind="dcsbm", blocks=3, edges=44300, alpha=1.5,
         draw_factor=1.011, feat="tfidf", feat_p=0.10, c0=500, classes=3, label="block",
         train=60, widths=[500, 128, 3], n_comm=16, n_iters=100),
    dict(name="powerlaw-large", n=169343, kind="dcsbm", blocks=40, edges=1170000, alpha=1.1,
         draw_factor=1.173, feat="normal", c0=128, classes=40, label="block",
         train_p=0.54, widths=[128, 256, 256, 40], n_comm=32, n_iters=50),
    dict(name="powerlaw-xlarge", n=2449029, kind="dcsbm", blocks=47, edges=61900000, alpha=1.0,
         draw_factor=1.222, feat="normal", c0=100, classes=47, label="block",
         train_p=0.08, widths=[100, 256, 256, 47], n_comm=64, n_iters=20),
    # shaped like the paper's own speed-up experiment (Section 4.1, Table 2): 13,752 nodes, 767 features,
    # 1000 hidden units, 10 classes, 1000 training nodes, 3 communities; the paper gives no edge count, so the
    # mean degree (30) and the feature density (0.3) are free choices made here
    dict(name="table2-shaped", n=13752, kind="dcsbm", blocks=10, edges=206280, alpha=1.5,
         draw_factor=1.068, feat="bow", feat_p=0.3, c0=767, classes=10, label="block",
         train=1000, widths=[767, 1000, 10], n_comm=3, n_iters=50),
]


def _symmetric_csr(n, u, v):
    """CSR (int64 row_ptr, int32 sorted col_idx) of the undirected simple graph with edges (u,v)."""
    keep = u != v
    u, v = u[keep], v[keep]
    rows = np.concatenate([u, v])
    cols = np.concatenate([v, u])
    A = sp.coo_matrix((np.ones(rows.shape[0], dtype=np.int32), (rows, cols)), shape=(n, n)).tocsr()
    A.sum_duplicates()
    A.sort_indices()
    return A.indptr.astype(np.int64), A.indices.astype(np.int32)


def _sbm_edges(rng, n, blocks, p_in, p_out):
    block = (np.arange(n) * blocks // n).astype(np.int32)
    iu, ju = np.triu_indices(n, k=1)
    p = np.where(block[iu] == block[ju], p_in, p_out)
    hit = rng.random(iu.shape[0]) < p
    return block, iu[hit], ju[hit]


def _dcsbm_edges(rng, n, blocks, n_edges, alpha, draw_factor):
    """Endpoints of a degree-corrected block model on ids whose blocks are contiguous."""
    block = (np.arange(n, dtype=np.int64) * blocks // n).astype(np.int32)
    mean_deg = 2.0 * n_edges / n
    w = rng.random(n) ** (-1.0 / alpha)
    cap_deg = math.sqrt(n * mean_deg)
    for _ in range(3):  # clip so that the expected degree 2|E| w_i / sum(w) stays below the cap
        w = np.minimum(w, cap_deg * w.sum() / (2.0 * n_edges))
    total = w.sum()
    starts = np.searchsorted(block, np.arange(blocks), side="left")
    ends = np.searchsorted(block, np.arange(blocks), side="right")
    n_draw = int(round(n_edges * draw_factor))
    # first endpoints ~ w, produced in ascending id order (the pairing below is what is random)
    u = np.repeat(np.arange(n, dtype=np.int64), rng.multinomial(n_draw, w / total))
    intra = rng.random(n_draw) < 0.85
    v = np.empty(n_draw, dtype=np.int64)
    u_lo = np.searchsorted(u, starts, side="left")
    u_hi = np.searchsorted(u, ends - 1, side="right")
    for b in range(blocks):  # second endpoints ~ w inside the block, shuffled against the first
        idx = u_lo[b] + np.flatnonzero(intra[u_lo[b]:u_hi[b]])
        wb = w[starts[b]:ends[b]]
        vb = np.repeat(np.arange(starts[b], ends[b], dtype=np.int64),
                       rng.multinomial(idx.shape[0], wb / wb.sum()))
        rng.shuffle(vb)
        v[idx] = vb
    idx = np.flatnonzero(~intra)   # the rest: second endpoints ~ w over all nodes
    vg = np.repeat(np.arange(n, dtype=np.int64), rng.multinomial(idx.shape[0], w / total))
    rng.shuffle(vg)
    v[idx] = vg
    return block, u, v


def _communities(n, row_ptr, col_idx, block, n_blocks, n_comm):
    if n_comm == n_blocks:
        return block.astype(np.int32).copy()
    deg = np.diff(row_ptr)
    A = sp.csr_matrix((np.ones(col_idx.shape[0], dtype=np.int8), col_idx, row_ptr), shape=(n, n))
    bfs = breadth_first_order(A, int(np.argmax(deg)), directed=False, return_predecessors=False)
    pos = np.full(n, n, dtype=np.int64)
    pos[bfs] = np.arange(bfs.shape[0])
    rest = np.flatnonzero(pos == n)
    pos[rest] = bfs.shape[0] + np.arange(rest.shape[0])
    order = np.lexsort((pos, block))
    community = np.empty(n, dtype=np.int32)
    community[order] = (np.arange(n, dtype=np.int64) * n_comm // n).astype(np.int32)
    return community


def glorot(rng, fan_in, fan_out):
    a = math.sqrt(6.0 / (fan_in + fan_out))
    return ((rng.random((fan_in, fan_out)) * 2.0 - 1.0) * a).astype(np.float32)


def make_workload(index: int, scale: float = 1.0, n_comm: int | None = None) -> Workload:
    """Build config ``index`` (0..5).  ``scale`` < 1 shrinks node and edge counts."""
    cfg = CONFIGS[index]
    rng = np.random.Generator(np.random.PCG64(BASE_SEED + index))
    n = max(int(round(cfg["n"] * scale)), 4 * cfg["blocks"])
    blocks = cfg["blocks"]
    if cfg["kind"] == "sbm":
        block, u, v = _sbm_edges(rng, n, blocks, cfg["p_in"], cfg["p_out"])
    else:
        n_edges = max(int(round(cfg["edges"] * n / cfg["n"])), n)
        block, u, v = _dcsbm_edges(rng, n, blocks, n_edges, cfg["alpha"], cfg["draw_factor"])
    # shuffle node ids so that blocks (and communities) are scattered in the original order
    relabel = rng.permutation(n).astype(np.int64)
    u = relabel[u]
    v = relabel[v]
    shuffled_block = np.empty(n, dtype=np.int32)
    shuffled_block[relabel] = block
    block = shuffled_block
    row_ptr, col_idx = _symmetric_csr(n, u, v)
    del u, v, relabel

    classes = cfg["classes"]
    if cfg["label"] == "noisy-block":
        primary = rng.integers(0, classes, size=blocks)
        keep = rng.random(n) < 0.8
        y = np.where(keep, primary[block], rng.integers(0, classes, size=n)).astype(np.int32)
    else:
        y = (block % classes).astype(np.int32)

    c0 = cfg["c0"]
    if cfg["feat"] == "bernoulli":
        X = (rng.random((n, c0)) < cfg["feat_p"]).astype(np.float32)
    elif cfg["feat"] == "bow":
        p = np.full((n, c0), cfg["feat_p"])
        seg = -(-c0 // classes)
        col_class = np.arange(c0) // seg
        p[y[:, None] == col_class[None, :]] *= 3.0
        X = (rng.random((n, c0)) < p).astype(np.float32)
    elif cfg["feat"] == "tfidf":
        nz = rng.random((n, c0)) < cfg["feat_p"]
        X = np.abs(rng.standard_normal((n, c0))) * nz
        X[np.arange(n), rng.integers(0, c0, size=n)] += 0.5  # no empty rows
        X = (X / np.linalg.norm(X, axis=1, keepdims=True)).astype(np.float32)
    else:
        X = rng.standard_normal((n, c0), dtype=np.float32)

    if "train" in cfg:
        n_train = max(int(round(cfg["train"] * n / cfg["n"])), 2 * classes)
        train_mask = np.zeros(n, dtype=np.uint8)
        train_mask[rng.choice(n, size=min(n_train, n), replace=False)] = 1
    else:
        train_mask = (rng.random(n) < cfg["train_p"]).astype(np.uint8)

    m = cfg["n_comm"] if n_comm is None else n_comm
    community = _communities(n, row_ptr, col_idx, block, blocks, m)
    widths = list(cfg["widths"])
    w_init = [glorot(rng, widths[l], widths[l + 1]) for l in range(len(widths) - 1)]
    return Workload(name=cfg["name"] if scale == 1.0 else f"{cfg['name']}@{scale:g}",
                    n=n, row_ptr=row_ptr, col_idx=col_idx, X=X, y=y, train_mask=train_mask,
                    widths=widths, n_comm=m, community=community, w_init=w_init,
                    n_iters=cfg["n_iters"], block=block)


def perturbed_state(wl: Workload, Z: list, seed: int, sigma: float = 0.1):
    """Gaussian perturbations (one per Z_l and one for U) used to leave the forward-consistent
    initial state, so that every term of every subproblem is active.  Returns float64 arrays
    ``dZ[l]`` shaped like ``Z[l]`` and ``dU`` shaped like ``Z[-1]``; the caller adds them."""
    rng = np.random.Generator(np.random.PCG64(seed))
    dZ = [sigma * rng.standard_normal(z.shape) for z in Z]
    dU = sigma * rng.standard_normal(Z[-1].shape)
    return dZ, dU
