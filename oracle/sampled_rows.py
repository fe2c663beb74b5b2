"""TEST INFRASTRUCTURE ONLY -- row-by-row fp64 evaluation of pieces of one ADMM pass.

For graphs on which the full oracle (``gcn_admm_oracle.OracleADMM``) cannot run a pass, the pieces
of a pass that are local to a row can still be computed exactly for a handful of sampled rows from
a given state: a row of A~ X, of the pre-activation H_l = A~ Z_{l-1} W_l, of the gradient of the
Z_{l,m} objective (Eq. 5 / Eq. 6; it needs the rows' neighbours and their neighbours), the
output-layer row of Eq. 7 and the dual row of Eq. 3.  Everything is taken straight from the CSR
pattern and the definitions; nothing is shared with the CUDA library.  ``tests/test_oracle_admm.py``
pins this file against the full oracle on small problems.
"""
from __future__ import annotations

import numpy as np


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
