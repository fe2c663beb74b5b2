"""TEST INFRASTRUCTURE ONLY -- plain fp64 CPU oracle of the community-based ADMM GCN trainer.

This file is the slow, by-the-book statement of what one ADMM iteration computes.  It is
used by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by
nothing else; it shares no code with the CUDA library and must never be imported by it.

Everything is numpy / scipy.sparse in float64, in the ORIGINAL node order, with explicit
index sets V_m per community.  No algebraic shortcut is taken: every subproblem objective
is evaluated from its printed definition each time it is needed (a full sparse product
and a full dense product per evaluation), every step size is found by sequential trials.

Where each function comes from (sections / equations of the paper):

* ``normalized_adjacency``        A~ = (D+I)^-1/2 (A+I) (D+I)^-1/2, Problem 1 text.
* ``community_index``             V_m, neighbour set N_m (Section 2), the block split of A~
                                  (Section 2) and the first / second order neighbour rows
                                  (Appendix A, first paragraph).
* ``forward``                     the constraints of Problem 1.
* ``OracleADMM.phi``              phi(W_l, Z_{l-1}, Z_l) and phi(W_L, Z_{L-1}, Z_L, U), Section 3.
* ``OracleADMM.update_W``         Section 3.1: quadratic approximation P_l(W; tau), the
                                  condition P_l(W^{k+1}; tau) >= phi(W^{k+1}), solution W - grad/tau.
* ``OracleADMM.psi``              Eq. (5) for l <= L-2 and Eq. (6) for l = L-1, Appendix A.
* ``OracleADMM.update_Z``         Eq. (8)-(10): Q_{l,m}(Z; theta), its condition and solution.
* ``OracleADMM.update_ZL``        Eq. (7), solved row by row with FISTA (Beck & Teboulle 2009).
* ``OracleADMM.update_U``         Eq. (3).
* ``OracleADMM.iterate``          Algorithm 1 (W blocks, then Z blocks, then U, all Jacobi).
* ``OracleADMM.iterate_sequential``  the serial schedule of Section 4.1 (one block after the other).
* ``OracleADMM.objective``        Eq. (1) in its full-graph form.
* ``OracleADMM.predict``          forward pass of Problem 1 with the current W.

Conventions the paper leaves open (the same ones the CUDA library documents; parity on these
is UNPINNED by the paper, they are stated choices):

* step parameters: each block keeps its tau / theta between iterations; a new search starts
  from max(previous * bt_shrink, 1e-12) and multiplies by bt_growth until the condition, in
  the reduced form f(x - g/t) <= f(x) - ||g||^2 / (2t), holds; at most bt_max_trials trials,
  after which the block is left unchanged and keeps its parameter; a block x whose gradient g
  has ||g||^2 <= 1e-24 ||x||^2 (zero up to rounding: the state right after the forward-pass
  initialisation) is skipped and keeps its parameter.
* risk: R = loss_scale * sum over training rows of the softmax cross-entropy; other rows add 0.
* activation: ReLU for l < L with derivative 1 for h > 0 and 0 otherwise; layer L is linear.
* FISTA for Eq. (7): the whole row objective is smooth, the non-smooth part is empty; constant
  step 1 / (loss_scale/2 + rho), t_1 = 1, warm start at the current row, exactly fista_iters
  iterations; rows outside the training mask take their exact minimiser q - u / rho.
* dual update: dual_mode 0 is Eq. (3) as printed (Z_L^k and Z_{L-1}^k with W_L^{k+1});
  dual_mode 1 is the textbook update with the k+1 iterates.
* initial state: given W, Z from the forward pass of Problem 1, U = 0, tau = tau0, theta = theta0.
* index lists are ascending and unique; nodes are ordered by (community, original id).
* serial schedule: block order W_1, Z_1, .., W_L, Z_L, U with the latest values everywhere (the paper only
  says that the layers are trained sequentially).
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import scipy.sparse as sp


@dataclass
class Params:
    nu: float = 1e-3
    rho: float = 1e-3
    tau0: float = 1.0
    theta0: float = 1.0
    bt_growth: float = 2.0
    bt_shrink: float = 0.5
    bt_max_trials: int = 40
    fista_iters: int = 30
    loss_scale: float = 1.0
    dual_mode: int = 0


SKIPPED = -1     # gradient (numerically) zero, block untouched
SKIP_REL2 = 1e-24  # a block x with ||grad||^2 <= SKIP_REL2 * ||x||^2 is skipped
EXHAUSTED = -2   # no trial met the condition, block untouched


# --------------------------------------------------------------------------------------
# graph side
# --------------------------------------------------------------------------------------

def normalized_adjacency(n, row_ptr, col_idx):
    """A~ = (D+I)^{-1/2} (A+I) (D+I)^{-1/2} as a scipy CSR matrix (Problem 1 text).

    ``row_ptr/col_idx`` is the CSR pattern of the undirected, unweighted A.  Diagonal entries
    of the input are ignored; exactly one identity is added.  D is the degree matrix of A."""
    row_ptr = np.asarray(row_ptr, dtype=np.int64)
    col_idx = np.asarray(col_idx, dtype=np.int64)
    rows = np.repeat(np.arange(n, dtype=np.int64), np.diff(row_ptr))
    off = rows != col_idx
    A = sp.csr_matrix((np.ones(int(off.sum())), (rows[off], col_idx[off])), shape=(n, n))
    A.data[:] = 1.0            # duplicates, if any, are not weights
    deg = np.asarray(A.sum(axis=1)).ravel()
    s = 1.0 / np.sqrt(deg + 1.0)
    At = sp.diags(s) @ (A + sp.identity(n, format="csr")) @ sp.diags(s)
    At = At.tocsr()
    At.sort_indices()
    return At


def community_index(n, row_ptr, col_idx, community, n_comm):
    """Index sets of the community split (Section 2; Appendix A, first paragraph).

    Returns a dict with, all int64 numpy arrays, ids in the NEW order (nodes sorted by
    (community, original id)):

    perm        new id -> original id          inv     original id -> new id
    comm_ptr    [M+1], V_m = new ids comm_ptr[m] .. comm_ptr[m+1]-1
    nbr[m]      N_m = { i != m : an edge joins V_m and V_i }, ascending
    halo1[m]    nodes outside V_m adjacent to a node of V_m (first-order neighbour rows)
    halo2[m]    nodes outside V_m and halo1[m] adjacent to a node of halo1[m] (second order)
    csr_row_ptr, csr_col   pattern of A+I in new ids, columns ascending
    seg_row_ptr [n+1], seg_comm [S], seg_begin [S+1]: row i owns segments
                seg_row_ptr[i] .. seg_row_ptr[i+1]-1; segment s covers positions
                seg_begin[s] .. seg_begin[s+1]-1 of csr_col, all of whose columns lie in
                community seg_comm[s] (this is row i of the block A~_{comm(i), seg_comm[s]}).
    """
    community = np.asarray(community, dtype=np.int64)
    row_ptr = np.asarray(row_ptr, dtype=np.int64)
    col_idx = np.asarray(col_idx, dtype=np.int64)
    perm = np.lexsort((np.arange(n), community))
    inv = np.empty(n, dtype=np.int64)
    inv[perm] = np.arange(n)
    comm_ptr = np.zeros(n_comm + 1, dtype=np.int64)
    comm_ptr[1:] = np.cumsum(np.bincount(community, minlength=n_comm))
    comm_new = community[perm]

    # adjacency sets in new ids, self loops removed, plus the single identity
    nbrs = []
    for i in range(n):
        o = perm[i]
        c = inv[col_idx[row_ptr[o]:row_ptr[o + 1]]]
        c = np.unique(np.concatenate([c[c != i], [i]]))
        nbrs.append(c)

    nbr, halo1, halo2 = [], [], []
    for m in range(n_comm):
        own = set(range(int(comm_ptr[m]), int(comm_ptr[m + 1])))
        h1 = set()
        for i in own:
            h1.update(int(j) for j in nbrs[i] if int(j) not in own)
        h2 = set()
        for j in h1:
            h2.update(int(k) for k in nbrs[j] if int(k) not in own and int(k) not in h1)
        halo1.append(np.array(sorted(h1), dtype=np.int64))
        halo2.append(np.array(sorted(h2), dtype=np.int64))
        nbr.append(np.array(sorted({int(comm_new[j]) for j in h1}), dtype=np.int64))

    csr_row_ptr = np.zeros(n + 1, dtype=np.int64)
    csr_row_ptr[1:] = np.cumsum([len(c) for c in nbrs])
    csr_col = np.concatenate(nbrs) if n else np.zeros(0, dtype=np.int64)
    seg_row_ptr = [0]
    seg_comm, seg_begin = [], []
    for i in range(n):
        base = int(csr_row_ptr[i])
        cc = comm_new[nbrs[i]]
        for k in range(len(cc)):
            if k == 0 or cc[k] != cc[k - 1]:
                seg_comm.append(int(cc[k]))
                seg_begin.append(base + k)
        seg_row_ptr.append(len(seg_comm))
    seg_begin.append(int(csr_row_ptr[n]))
    return dict(perm=perm, inv=inv, comm_ptr=comm_ptr, nbr=nbr, halo1=halo1, halo2=halo2,
                csr_row_ptr=csr_row_ptr, csr_col=csr_col,
                seg_row_ptr=np.array(seg_row_ptr, dtype=np.int64),
                seg_comm=np.array(seg_comm, dtype=np.int64),
                seg_begin=np.array(seg_begin, dtype=np.int64))


# --------------------------------------------------------------------------------------
# network side
# --------------------------------------------------------------------------------------

def relu(h):
    return np.maximum(h, 0.0)


def relu_grad(h):
    return (h > 0.0).astype(np.float64)


def forward(At, X, W):
    """Z_l = f_l(A~ Z_{l-1} W_l) for l < L and Z_L = A~ Z_{L-1} W_L (constraints of Problem 1).
    ``W`` is the list W_1..W_L; returns [Z_0, Z_1, .., Z_L]."""
    Z = [np.asarray(X, dtype=np.float64)]
    L = len(W)
    for l in range(1, L + 1):
        H = (At @ Z[l - 1]) @ W[l - 1]
        Z.append(relu(H) if l < L else H)
    return Z


def cross_entropy_rows(Z, y):
    """-log softmax(Z[i])[y[i]] per row."""
    zmax = Z.max(axis=1, keepdims=True)
    lse = zmax[:, 0] + np.log(np.exp(Z - zmax).sum(axis=1))
    return lse - Z[np.arange(Z.shape[0]), y]


def softmax_rows(Z):
    e = np.exp(Z - Z.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


class OracleADMM:
    """State and block updates of Algorithm 1.  Lists are 1-based in the layer index: ``W[l]``,
    ``Z[l]``, ``tau[l]`` for l = 1..L (``Z[0]`` is the feature matrix); ``theta[l][m]``."""

    def __init__(self, n, row_ptr, col_idx, X, y, train_mask, widths, params, n_comm, community,
                 w_init):
        self.n = int(n)
        self.p = params
        self.L = len(widths) - 1
        self.widths = list(widths)
        self.M = int(n_comm)
        self.forced_tol = 1e-6    # replay mode: slack on the condition q >= 1 of a forced trial
        self.At = normalized_adjacency(n, row_ptr, col_idx)
        self.y = np.asarray(y, dtype=np.int64)
        self.train = np.asarray(train_mask).astype(bool)
        community = np.asarray(community, dtype=np.int64)
        self.community = community
        self.V = [np.flatnonzero(community == m) for m in range(self.M)]
        # N_m from its definition: communities i != m joined to V_m by an edge
        pattern = self.At.copy()
        pattern.setdiag(0.0)
        pattern.eliminate_zeros()
        coo = pattern.tocoo()
        cu, cv = community[coo.row], community[coo.col]
        self.nbr = [np.unique(cv[(cu == m) & (cv != m)]) for m in range(self.M)]
        # rows on which psi_m of Eq. (5)/(6) is evaluated: V_m, then every V_r with r in N_m
        self.rows_ext = [np.concatenate([self.V[m]] + [self.V[r] for r in self.nbr[m]])
                         for m in range(self.M)]
        self.At_ext = [self.At[rows, :] for rows in self.rows_ext]
        self.W = [None] + [np.array(w, dtype=np.float64) for w in w_init]
        self.Z = forward(self.At, X, self.W[1:])
        self.U = np.zeros_like(self.Z[self.L])
        self.tau = [None] + [float(params.tau0)] * self.L
        self.theta = [None] + [[float(params.theta0)] * self.M for _ in range(1, self.L)]
        for l in range(1, self.L + 1):
            assert self.W[l].shape == (widths[l - 1], widths[l])

    # ---- activations per layer --------------------------------------------------------
    def f(self, l, h):
        return relu(h) if l < self.L else h

    # ---- W blocks (Section 3.1) -------------------------------------------------------
    def phi(self, l, Wl, Z=None, U=None):
        """phi(W_l, Z_{l-1}, Z_l) for l < L; phi(W_L, Z_{L-1}, Z_L, U) for l = L (Section 3)."""
        Z = self.Z if Z is None else Z
        U = self.U if U is None else U
        H = (self.At @ Z[l - 1]) @ Wl
        if l < self.L:
            return 0.5 * self.p.nu * np.sum((Z[l] - relu(H)) ** 2)
        r = Z[l] - H
        return np.sum(U * r) + 0.5 * self.p.rho * np.sum(r * r)

    def grad_phi(self, l, Wl=None, Z=None, U=None):
        Z = self.Z if Z is None else Z
        U = self.U if U is None else U
        Wl = self.W[l] if Wl is None else Wl
        P = self.At @ Z[l - 1]
        H = P @ Wl
        if l < self.L:
            return self.p.nu * (P.T @ ((relu(H) - Z[l]) * relu_grad(H)))
        return -(P.T @ (U + self.p.rho * (Z[l] - H)))

    def _search(self, fun, x, g, t_prev, forced):
        """Sequential search for the step parameter t of a quadratic-approximation step
        x+ = x - g / t under the condition fun(x+) <= fun(x) - ||g||^2 / (2 t).

        The record holds the accepted trial index, t, ``q`` = (fun(x) - fun(x+)) / (||g||^2/(2t))
        at the accepted trial (the condition reads q >= 1), ``q_reject`` at the last rejected
        trial, and ``margin`` = min(|q - 1|, |q_reject - 1|): how far the decision was from a tie."""
        p = self.p
        gg = float(np.sum(g * g))
        if gg <= SKIP_REL2 * float(np.sum(x * x)):
            return x, t_prev, dict(trial=SKIPPED, t=t_prev, margin=np.inf, gg=gg, ok=True)
        f0 = float(fun(x))
        t = max(t_prev * p.bt_shrink, 1e-12)
        if forced is not None:
            if forced < 0:
                return x, t_prev, dict(trial=int(forced), t=t_prev, margin=0.0, gg=gg, ok=True)
            t = t * p.bt_growth ** forced
            xn = x - g / t
            q = (f0 - float(fun(xn))) / (gg / (2.0 * t))
            q_prev = -np.inf          # the trial before the forced one must not have passed
            if forced > 0:
                tp = t / p.bt_growth
                q_prev = (f0 - float(fun(x - g / tp))) / (gg / (2.0 * tp))
            tol = self.forced_tol
            return xn, t, dict(trial=int(forced), t=t, q=q, q_reject=q_prev, gg=gg, f0=f0,
                               margin=min(abs(q - 1.0), abs(q_prev - 1.0)),
                               ok=bool(q >= 1.0 - tol and q_prev < 1.0 + tol))
        q_reject = np.inf
        for trial in range(p.bt_max_trials):
            xn = x - g / t
            f1 = float(fun(xn))
            q = (f0 - f1) / (gg / (2.0 * t))
            if f1 <= f0 - gg / (2.0 * t):
                return xn, t, dict(trial=trial, t=t, q=q, q_reject=q_reject, gg=gg, ok=True, f0=f0,
                                   f1=f1, margin=min(abs(q - 1.0), abs(q_reject - 1.0)))
            q_reject = q
            t *= p.bt_growth
        return x, t_prev, dict(trial=EXHAUSTED, t=t_prev, margin=abs(q_reject - 1.0), gg=gg, ok=False)

    def update_W(self, l, forced=None, Z=None, U=None):
        """W_l^{k+1} = W_l^k - grad / tau_l^{k+1} (Section 3.1).  Returns (W_new, record)."""
        g = self.grad_phi(l, Z=Z, U=U)
        Wn, t, rec = self._search(lambda w: self.phi(l, w, Z=Z, U=U), self.W[l], g, self.tau[l],
                                  forced)
        return Wn, t, rec

    # ---- hidden Z blocks (Appendix A, Eq. (5), (6), (8)-(10)) -------------------------
    def psi(self, l, m, Zlm, W=None, Z=None, U=None):
        """Objective of Z_{l,m} for 1 <= l <= L-1: Eq. (5) when l <= L-2, Eq. (6) when l = L-1.

        The sums over r of first-order messages p_{l,r->m} and the second-order pieces
        s_{l,r->m} are formed together as rows of A~ Z_l' W_{l+1}, where Z_l' is Z_l^k with
        the rows of community m replaced by the argument."""
        W = self.W if W is None else W
        Z = self.Z if Z is None else Z
        U = self.U if U is None else U
        p, L = self.p, self.L
        Vm = self.V[m]
        pre_l = (self.At[Vm, :] @ Z[l - 1]) @ W[l]              # sum_r p_{l-1, r->m}
        total = 0.5 * p.nu * np.sum((Zlm - relu(pre_l)) ** 2)
        Zl = Z[l].copy()
        Zl[Vm] = Zlm
        rows = self.rows_ext[m]                                 # V_m and V_r, r in N_m
        pre = (self.At_ext[m] @ Zl) @ W[l + 1]
        if l + 1 < L:
            total += 0.5 * p.nu * np.sum((Z[l + 1][rows] - relu(pre)) ** 2)
        else:
            res = Z[L][rows] - pre
            total += np.sum(U[rows] * res) + 0.5 * p.rho * np.sum(res * res)
        return total

    def grad_psi(self, l, m, W=None, Z=None, U=None):
        """Gradient of ``psi`` with respect to Z_{l,m} at Z_{l,m}^k."""
        W = self.W if W is None else W
        Z = self.Z if Z is None else Z
        U = self.U if U is None else U
        p, L = self.p, self.L
        Vm = self.V[m]
        pre_l = (self.At[Vm, :] @ Z[l - 1]) @ W[l]
        g = p.nu * (Z[l][Vm] - relu(pre_l))
        for r in [m] + list(self.nbr[m]):
            Vr = self.V[r]
            pre = (self.At[Vr, :] @ Z[l]) @ W[l + 1]
            if l + 1 < L:
                back = p.nu * (relu(pre) - Z[l + 1][Vr]) * relu_grad(pre)
            else:
                back = -(U[Vr] + p.rho * (Z[L][Vr] - pre))
            A_rm = self.At[Vr, :][:, Vm]
            g = g + (A_rm.T @ back) @ W[l + 1].T
        return g

    def update_Z(self, l, m, W, forced=None, Z=None, U=None):
        """Z_{l,m}^{k+1} = Z_{l,m}^k - grad psi / theta_{l,m}^{k+1}, Eq. (10), for l < L."""
        Zs = self.Z if Z is None else Z
        g = self.grad_psi(l, m, W=W, Z=Z, U=U)
        Zn, t, rec = self._search(lambda z: self.psi(l, m, z, W=W, Z=Z, U=U), Zs[l][self.V[m]], g,
                                  self.theta[l][m], forced)
        return Zn, t, rec

    # ---- output layer (Eq. (7)) -------------------------------------------------------
    def psi_L_rows(self, Zrows, q, u, y, train):
        """Row-wise value of the Eq. (7) objective (it is separable by row)."""
        p = self.p
        val = np.sum(u * (Zrows - q), axis=1) + 0.5 * p.rho * np.sum((Zrows - q) ** 2, axis=1)
        ce = cross_entropy_rows(Zrows, y)
        return val + np.where(train, p.loss_scale * ce, 0.0)

    def grad_psi_L_rows(self, Zrows, q, u, y):
        p = self.p
        sm = softmax_rows(Zrows)
        sm[np.arange(Zrows.shape[0]), y] -= 1.0
        return p.loss_scale * sm + u + p.rho * (Zrows - q)

    def update_ZL(self, W, Z=None, U=None, iters=None):
        """Z_L^{k+1}: Eq. (7).  q = (A~ Z_{L-1}^k W_L^{k+1}); training rows by FISTA, the
        others by their exact minimiser q - u / rho."""
        Z = self.Z if Z is None else Z
        U = self.U if U is None else U
        p, L = self.p, self.L
        iters = p.fista_iters if iters is None else iters
        q = (self.At @ Z[L - 1]) @ W[L]
        Zn = q - U / p.rho
        tr = np.flatnonzero(self.train)
        if tr.size:
            qt, ut, yt = q[tr], U[tr], self.y[tr]
            step = 1.0 / (0.5 * p.loss_scale + p.rho)
            x_prev = Z[L][tr].copy()
            v = x_prev.copy()
            t = 1.0
            for _ in range(iters):
                x = v - step * self.grad_psi_L_rows(v, qt, ut, yt)
                t_next = 0.5 * (1.0 + np.sqrt(1.0 + 4.0 * t * t))
                v = x + ((t - 1.0) / t_next) * (x - x_prev)
                x_prev, t = x, t_next
            Zn[tr] = x_prev
        return Zn

    # ---- dual (Eq. (3)) ---------------------------------------------------------------
    def update_U(self, W, Z_for_dual, U=None):
        """U + rho (Z_L - A~ Z_{L-1} W_L) with the iterates handed in (Eq. (3))."""
        U = self.U if U is None else U
        L = self.L
        return U + self.p.rho * (Z_for_dual[L] - (self.At @ Z_for_dual[L - 1]) @ W[L])

    # ---- Algorithm 1 ------------------------------------------------------------------
    def iterate(self, forced=None):
        """One pass of Algorithm 1.  ``forced`` optionally fixes the accepted trial of each block:
        dict with 'W': {l: trial} and 'Z': {(l, m): trial}.  Returns the record of decisions."""
        L, M = self.L, self.M
        rec = dict(W={}, Z={})
        fW = (forced or {}).get("W", {})
        fZ = (forced or {}).get("Z", {})
        Wn, taun = list(self.W), list(self.tau)
        for l in range(1, L + 1):                      # every W_l from (W^k, Z^k, U^k)
            Wn[l], taun[l], rec["W"][l] = self.update_W(l, forced=fW.get(l))
        Zn = [z for z in self.Z]
        thetan = [None] + [list(t) for t in self.theta[1:]]
        for l in range(1, L):                          # every Z_{l,m} from (W^{k+1}, Z^k, U^k)
            Zl = self.Z[l].copy()
            for m in range(M):
                Zlm, thetan[l][m], rec["Z"][(l, m)] = self.update_Z(l, m, Wn, forced=fZ.get((l, m)))
                Zl[self.V[m]] = Zlm
            Zn[l] = Zl
        Zn[L] = self.update_ZL(Wn)
        if self.p.dual_mode == 0:                      # dual update, Eq. (3) as printed
            Un = self.update_U(Wn, self.Z)
        else:
            Un = self.update_U(Wn, Zn)
        self.W, self.tau, self.Z, self.theta, self.U = Wn, taun, Zn, thetan, Un
        return rec

    def iterate_sequential(self, forced=None, trace=None):
        """The serial schedule of Section 4.1 ("layers trained sequentially"): the same block updates as
        Algorithm 1, but taken one after the other in the order W_1, Z_1, W_2, Z_2, .., W_L, Z_L, U, each
        reading the latest value of every other block (the communities of one layer still move together,
        from the same Z_l).  ``trace``, when a list, receives L_rho after every block."""
        L, M = self.L, self.M
        rec = dict(W={}, Z={})
        fW = (forced or {}).get("W", {})
        fZ = (forced or {}).get("Z", {})
        for l in range(1, L + 1):
            self.W[l], self.tau[l], rec["W"][l] = self.update_W(l, forced=fW.get(l))
            if trace is not None:
                trace.append(("W", l, self.objective()[0]))
            if l < L:
                Zl = self.Z[l].copy()
                for m in range(M):
                    Zlm, self.theta[l][m], rec["Z"][(l, m)] = self.update_Z(l, m, self.W, forced=fZ.get((l, m)))
                    Zl[self.V[m]] = Zlm
                self.Z[l] = Zl
            else:
                self.Z[L] = self.update_ZL(self.W)
            if trace is not None:
                trace.append(("Z", l, self.objective()[0]))
        self.U = self.update_U(self.W, self.Z)
        return rec

    # ---- reporting --------------------------------------------------------------------
    def objective(self):
        """[L_rho, R, sum_l phi_l (l<L), <U, r>, rho/2 ||r||^2, train accuracy], Eq. (1)."""
        p, L = self.p, self.L
        tr = np.flatnonzero(self.train)
        R = p.loss_scale * float(np.sum(cross_entropy_rows(self.Z[L][tr], self.y[tr]))) if tr.size else 0.0
        pen = sum(float(self.phi(l, self.W[l])) for l in range(1, L))
        r = self.Z[L] - (self.At @ self.Z[L - 1]) @ self.W[L]
        ur = float(np.sum(self.U * r))
        rr = 0.5 * p.rho * float(np.sum(r * r))
        _, labels = self.predict()
        acc = float(np.mean(labels[tr] == self.y[tr])) if tr.size else 0.0
        return np.array([R + pen + ur + rr, R, pen, ur, rr, acc])

    def predict(self):
        """Logits of the forward pass of Problem 1 with the current W, and their row argmax
        (ties to the lowest class index)."""
        logits = forward(self.At, self.Z[0], self.W[1:])[self.L]
        return logits, np.argmax(logits, axis=1)
