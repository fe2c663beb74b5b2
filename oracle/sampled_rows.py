"""TEST INFRASTRUCTURE ONLY -- row-by-row fp64 evaluation of pieces of one ADMM pass.

For graphs on which the full oracle (``gcn_admm_oracle.OracleADMM``) cannot run a pass, the pieces
of a pass that are local to a row can still be computed exactly for a handful of sampled rows from
a given state: a row of A~ X, of the pre-activation H_l = A~ Z_{l-1} W_l, of the gradient of the
Z_{l,m} objective (Eq. 5 / Eq. 6; it needs the rows' neighbours and their neighbours), the
output-layer row of Eq. 7 and the dual row of Eq. 3.  One community's step-size decision can be
checked the same way: the change of its objective psi_m (Eq. 5 / Eq. 6) along the step of Eq. 10 needs
only the community's rows and the rows adjacent to them (``psi_change``), so the condition of Eq. 9 can
be evaluated in fp64 for a sampled community of a graph of any size.  Everything is taken straight from
the CSR pattern and the definitions; nothing is shared with the CUDA library.  ``tests/test_oracle_admm.py``
pins this file against the full oracle on small problems.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import scipy.sparse as sp


class SampledRows:
    def __init__(self, n, row_ptr, col_idx, y, train_mask, widths, nu, rho, loss_scale=1.0, fista_iters=30):
        self.n = int(n)
        self.row_ptr = np.asarray(row_ptr, dtype=np.int64)
        self.col_idx = np.asarray(col_idx)
        self.L = len(widths) - 1
        self.nu, self.rho, self.loss_scale, self.fista_iters = float(nu), float(rho), float(loss_scale), int(fista_iters)
        self.y = np.asarray(y)
        self.train = np.asarray(train_mask).astype(bool)
        deg = np.diff(self.row_ptr).astype(np.float64)
        # input self loops do not count towards the degree (Problem 1: D is the degree matrix of A)
        rows = np.repeat(np.arange(self.n), np.diff(self.row_ptr))
        deg -= np.bincount(rows[self.col_idx == rows], minlength=self.n)
        self.d = deg + 1.0

    def adj_row(self, i):
        """Columns and values of row i of A~ = (D+I)^-1/2 (A+I) (D+I)^-1/2."""
        c = np.asarray(self.col_idx[self.row_ptr[i]:self.row_ptr[i + 1]], dtype=np.int64)
        c = np.unique(np.concatenate([c[c != i], [i]]))
        return c, 1.0 / np.sqrt(self.d[i] * self.d[c])

    def propagate_rows(self, X, rows):
        out = np.zeros((len(rows), X.shape[1]))
        for k, i in enumerate(rows):
            c, v = self.adj_row(int(i))
            out[k] = v @ np.asarray(X[c], dtype=np.float64)
        return out

    def H_rows(self, l, rows, Z, W):
        """Rows of A~ Z_{l-1} W_l.  Z[0] is the feature matrix; W[l], Z[l] are 1-based lists."""
        return self.propagate_rows(Z[l - 1], rows) @ np.asarray(W[l], dtype=np.float64)

    def back_rows(self, l, rows, Z, W, U):
        """Derivative of the layer-l term with respect to H_l at the given rows:
        nu (f(H) - Z_l) f'(H) for l < L, -(U + rho (Z_L - H)) for l = L."""
        H = self.H_rows(l, rows, Z, W)
        Zl = np.asarray(Z[l][rows], dtype=np.float64)
        if l < self.L:
            return self.nu * (np.maximum(H, 0.0) - Zl) * (H > 0.0)
        return -(np.asarray(U[rows], dtype=np.float64) + self.rho * (Zl - H))

    def grad_Z_rows(self, l, rows, Z, W, U):
        """Rows of the gradient of psi (Eq. 5 for l <= L-2, Eq. 6 for l = L-1) with respect to Z_l:
        nu (Z_l - f(H_l)) + sum_j A~_ij back_{l+1}[j] W_{l+1}^T  (A~ is symmetric)."""
        out = np.zeros((len(rows), Z[l].shape[1]))
        Wn = np.asarray(W[l + 1], dtype=np.float64)
        for k, i in enumerate(rows):
            i = int(i)
            H = self.H_rows(l, [i], Z, W)[0]
            g = self.nu * (np.asarray(Z[l][i], dtype=np.float64) - np.maximum(H, 0.0))
            c, v = self.adj_row(i)
            back = self.back_rows(l + 1, c, Z, W, U)
            out[k] = g + (v @ back) @ Wn.T
        return out

    def ZL_rows(self, rows, Z, W, U):
        """Rows of the Eq. 7 update: q - u/rho off the training set, FISTA on it."""
        L, rho, s = self.L, self.rho, self.loss_scale
        q = self.H_rows(L, rows, Z, W)
        u = np.asarray(U[rows], dtype=np.float64)
        out = q - u / rho
        step = 1.0 / (0.5 * s + rho)
        for k, i in enumerate(rows):
            if not self.train[i]:
                continue
            x_prev = np.asarray(Z[L][i], dtype=np.float64).copy()
            v = x_prev.copy()
            t = 1.0
            for _ in range(self.fista_iters):
                e = np.exp(v - v.max())
                p = e / e.sum()
                p[self.y[i]] -= 1.0
                x = v - step * (s * p + u[k] + rho * (v - q[k]))
                tn = 0.5 * (1.0 + np.sqrt(1.0 + 4.0 * t * t))
                v = x + ((t - 1.0) / tn) * (x - x_prev)
                x_prev, t = x, tn
            out[k] = x_prev
        return out

    def U_rows(self, rows, Z, W, U):
        """Rows of U + rho (Z_L - A~ Z_{L-1} W_L), Eq. 3."""
        L = self.L
        return np.asarray(U[rows], dtype=np.float64) + self.rho * (np.asarray(Z[L][rows], dtype=np.float64) -
                                                                  self.H_rows(L, rows, Z, W))


    # ---- one community's step-size condition (Eq. 8-10) -------------------------------------------
    def adj_rows(self, rows):
        """Rows ``rows`` of A~ as a scipy CSR matrix of shape (len(rows), n), fp64."""
        rows = np.asarray(rows, dtype=np.int64)
        start, stop = self.row_ptr[rows], self.row_ptr[rows + 1]
        cnt = stop - start
        local = np.repeat(np.arange(rows.shape[0], dtype=np.int64), cnt)
        pos = np.arange(int(cnt.sum()), dtype=np.int64) - np.repeat(np.cumsum(cnt) - cnt, cnt) + np.repeat(start, cnt)
        cols = np.asarray(self.col_idx[pos], dtype=np.int64)
        keep = cols != rows[local]                     # input self loops are dropped, one identity is added
        local = np.concatenate([local[keep], np.arange(rows.shape[0], dtype=np.int64)])
        cols = np.concatenate([cols[keep], rows])
        vals = 1.0 / np.sqrt(self.d[rows[local]] * self.d[cols])
        A = sp.csr_matrix((vals, (local, cols)), shape=(rows.shape[0], self.n))
        A.sort_indices()
        return A

    @staticmethod
    def _times(A, X, block=32):
        """A @ X in fp64 for a dense X of any float type, a block of columns at a time (X may be large; the
        blocks are independent, so they are handed to a few threads -- the arithmetic is unchanged)."""
        out = np.empty((A.shape[0], X.shape[1]))

        def one(c):
            out[:, c:c + block] = A @ np.asarray(X[:, c:c + block], dtype=np.float64)
        with ThreadPoolExecutor(max_workers=min(os.cpu_count() or 1, 16)) as pool:
            list(pool.map(one, range(0, X.shape[1], block)))
        return out

    def psi_change(self, l, Vm, Z, W, U, thetas):
        """For the community with node set ``Vm`` and hidden layer l (1 <= l <= L-1), at the state (Z, W, U):
        ``gg`` = ||grad psi_m||^2 and, for every theta in ``thetas``, psi_m(Z_{l,m} - grad/theta) - psi_m(Z_{l,m})
        with psi_m of Eq. 5 (l <= L-2) or Eq. 6 (l = L-1).  Only rows of V_m and rows adjacent to V_m enter:
        every other row of a neighbouring community adds the same constant to both values of psi_m.
        The condition of Eq. 9 at theta, in the form the step of Eq. 10 gives it, reads
        -change >= gg / (2 theta)."""
        L, nu, rho = self.L, self.nu, self.rho
        Vm = np.sort(np.asarray(Vm, dtype=np.int64))
        Am = self.adj_rows(Vm)                                     # |V_m| x n
        ext = np.unique(Am.indices.astype(np.int64))               # V_m and its first-order neighbour rows
        Ae = self.adj_rows(ext)                                    # |ext| x n
        Wl, Wn = np.asarray(W[l], dtype=np.float64), np.asarray(W[l + 1], dtype=np.float64)
        Zm = np.asarray(Z[l][Vm], dtype=np.float64)
        fH = np.maximum(self._times(Am, Z[l - 1]) @ Wl, 0.0)       # f_l(H_l) on V_m
        Hn = self._times(Ae, Z[l]) @ Wn                            # H_{l+1} on ext
        Zn = np.asarray(Z[l + 1][ext], dtype=np.float64)
        if l + 1 < L:
            back = nu * (np.maximum(Hn, 0.0) - Zn) * (Hn > 0.0)
        else:
            Ue = np.asarray(U[ext], dtype=np.float64)
            back = -(Ue + rho * (Zn - Hn))
        G = nu * (Zm - fH) + (Am[:, ext] @ back) @ Wn.T            # grad of psi_m w.r.t. Z_{l,m} (A~ symmetric)
        gg = float(np.sum(G * G))
        K = Ae[:, Vm] @ (G @ Wn)                                   # change of H_{l+1} on ext per unit 1/theta

        def next_term(H):
            if l + 1 < L:
                return 0.5 * nu * np.sum((Zn - np.maximum(H, 0.0)) ** 2)
            r = Zn - H
            return np.sum(Ue * r) + 0.5 * rho * np.sum(r * r)

        base = 0.5 * nu * np.sum((Zm - fH) ** 2) + next_term(Hn)
        out = []
        for t in thetas:
            Zt = Zm - G / t
            out.append(float(0.5 * nu * np.sum((Zt - fH) ** 2) + next_term(Hn - K / t) - base))
        return gg, out
