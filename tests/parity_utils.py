"""Helpers shared by the GPU parity tests: build the CUDA handle and the fp64 oracle from one
seeded workload, put both in the same state, compare."""
import numpy as np

from oracle import gcn_admm_oracle as orc
from paper_2112_09335_b200 import binding


def make_oracle(wl, **params):
    kw = dict(nu=wl.nu, rho=wl.rho)
    kw.update(params)
    return orc.OracleADMM(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, orc.Params(**kw),
                          wl.n_comm, wl.community, wl.w_init)


def make_pair(wl, **params):
    """(GcnAdmm handle, OracleADMM) on the same workload and parameters."""
    kw = dict(nu=wl.nu, rho=wl.rho)
    kw.update(params)
    g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                        wl.w_init, **kw)
    return g, make_oracle(wl, **params)


def relerr(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / d) if d > 0 else float(np.linalg.norm(a - b))


def push_state(g, o, Z=None, U=None, W=None, tau=None, theta=None):
    """Writes a state into both sides.  Values are rounded to fp32 first so that the two start
    from bit-identical numbers."""
    L = o.L
    if W is not None:
        for l in range(1, L + 1):
            w32 = np.asarray(W[l], dtype=np.float32)
            g.set_state(binding.ST_W, l, w32)
            o.W[l] = w32.astype(np.float64)
    if Z is not None:
        for l in range(1, L + 1):
            z32 = np.asarray(Z[l], dtype=np.float32)
            g.set_state(binding.ST_Z, l, z32)
            o.Z[l] = z32.astype(np.float64)
    if U is not None:
        u32 = np.asarray(U, dtype=np.float32)
        g.set_state(binding.ST_U, 0, u32)
        o.U = u32.astype(np.float64)
    if tau is not None:
        for l in range(1, L + 1):
            g.set_state(binding.ST_TAU, l, np.array([tau[l]]))
            o.tau[l] = float(tau[l])
    if theta is not None:
        for l in range(1, L):
            g.set_state(binding.ST_THETA, l, np.asarray(theta[l], dtype=np.float64))
            o.theta[l] = [float(t) for t in theta[l]]


def forced_from(dec, k, L, M):
    """Decisions of GPU pass k as the oracle's ``forced`` argument."""
    return dict(W={l: int(dec["trial_w"][k, l - 1]) for l in range(1, L + 1)},
                Z={(l, m): int(dec["trial_z"][k, l - 1, m]) for l in range(1, L) for m in range(M)})


def compare_decisions(rec, dec, k, L, M):
    """Lists the blocks whose accepted trial differs between an oracle record and GPU pass k,
    with the oracle's distance from a tie."""
    out = []
    for l in range(1, L + 1):
        if rec["W"][l]["trial"] != dec["trial_w"][k, l - 1]:
            out.append((("W", l), rec["W"][l]["trial"], int(dec["trial_w"][k, l - 1]), rec["W"][l]["margin"]))
    for l in range(1, L):
        for m in range(M):
            r = rec["Z"][(l, m)]
            if r["trial"] != dec["trial_z"][k, l - 1, m]:
                out.append((("Z", l, m), r["trial"], int(dec["trial_z"][k, l - 1, m]), r["margin"]))
    return out
