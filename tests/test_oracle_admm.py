"""Pins of the oracle's ADMM side.  Each check uses something the oracle does not: dense
matrices, the per-community message form printed in the paper, central finite differences,
an eigen-solve, a Newton solve, or an exact special case."""
import numpy as np
import pytest

from conftest import tiny_problem
from oracle import gcn_admm_oracle as orc


def make(seed, perturb=0.3, **kw):
    params = orc.Params(nu=kw.pop("nu", 0.7), rho=kw.pop("rho", 0.9))
    pr = tiny_problem(seed, **kw)
    o = orc.OracleADMM(pr["n"], pr["row_ptr"], pr["col_idx"], pr["X"], pr["y"], pr["mask"],
                       pr["widths"], params, pr["n_comm"], pr["community"], pr["W"])
    if perturb:
        rng = np.random.default_rng(seed + 1000)
        for l in range(1, o.L + 1):
            o.Z[l] = o.Z[l] + perturb * rng.standard_normal(o.Z[l].shape)
        o.U = perturb * rng.standard_normal(o.U.shape)
    return pr, o


def dense_At(pr):
    A = pr["A"]
    d = A.sum(axis=1) + 1.0
    return (A + np.eye(pr["n"])) / np.sqrt(np.outer(d, d))


def keep_off_kinks(o, margin=1e-3):
    """True when every hidden pre-activation is at least ``margin`` away from the ReLU kink."""
    for l in range(1, o.L):
        H = (o.At @ o.Z[l - 1]) @ o.W[l]
        if np.abs(H).min() < margin:
            return False
    return True


def num_grad(f, x, h=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        xp, xm = x.copy(), x.copy()
        xp[i] += h
        xm[i] -= h
        g[i] = (f(xp) - f(xm)) / (2 * h)
    return g


# ---- the paper's per-community message form, written with dense blocks ------------------

def psi_message_form(pr, o, l, m, Zlm):
    """Eq. (5) / Eq. (6) exactly as printed: first-order messages p, second-order s = [s1, s2],
    blocks A~_{a,b} cut out of a dense matrix."""
    At = dense_At(pr)
    L, nu, rho = o.L, o.p.nu, o.p.rho
    V = [np.flatnonzero(pr["community"] == c) for c in range(pr["n_comm"])]
    Nm = lambda c: [r for r in range(pr["n_comm"]) if r != c and At[np.ix_(V[c], V[r])].any()]
    blk = lambda a, b: At[np.ix_(V[a], V[b])]
    relu = lambda h: np.maximum(h, 0)
    p = lambda lay, r, c: blk(c, r) @ o.Z[lay][V[r]] @ o.W[lay + 1]     # p_{lay, r->c}
    total = 0.5 * nu * np.sum((Zlm - relu(sum(p(l - 1, r, m) for r in Nm(m) + [m]))) ** 2)
    own_pre = blk(m, m) @ Zlm @ o.W[l + 1] + sum([p(l, r, m) for r in Nm(m)], 0)
    if l + 1 < L:
        total += 0.5 * nu * np.sum((o.Z[l + 1][V[m]] - relu(own_pre)) ** 2)
    else:
        res = o.Z[L][V[m]] - own_pre
        total += np.sum(o.U[V[m]] * res) + 0.5 * rho * np.sum(res ** 2)
    for r in Nm(m):
        others = [q for q in Nm(r) + [r] if q != m]
        agg = sum([p(l, q, r) for q in others], 0)                     # what r aggregates
        if l + 1 < L:
            s1, s2 = o.Z[l + 1][V[r]], agg
            total += 0.5 * nu * np.sum((s1 - relu(blk(r, m) @ Zlm @ o.W[l + 1] + s2)) ** 2)
        else:
            s1, s2 = o.Z[L][V[r]] - agg, o.U[V[r]]
            res = s1 - blk(r, m) @ Zlm @ o.W[L]
            total += np.sum(s2 * res) + 0.5 * rho * np.sum(res ** 2)
    return total


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_psi_equals_printed_message_form(seed):
    pr, o = make(seed)
    rng = np.random.default_rng(seed)
    for l in range(1, o.L):
        for m in range(o.M):
            Zlm = o.Z[l][o.V[m]] + 0.2 * rng.standard_normal((len(o.V[m]), o.widths[l]))
            a = o.psi(l, m, Zlm)
            b = psi_message_form(pr, o, l, m, Zlm)
            assert abs(a - b) <= 1e-12 * max(1.0, abs(b))


@pytest.mark.parametrize("seed", [0, 3])
def test_phi_full_graph_equals_community_sum(seed):
    """phi in its per-community form (Section 3) equals the full-graph form."""
    pr, o = make(seed)
    At = dense_At(pr)
    V = o.V
    for l in range(1, o.L + 1):
        total = 0.0
        for m in range(o.M):
            pre = sum(At[np.ix_(V[m], V[r])] @ o.Z[l - 1][V[r]] for r in range(o.M)) @ o.W[l]
            if l < o.L:
                total += 0.5 * o.p.nu * np.sum((o.Z[l][V[m]] - np.maximum(pre, 0)) ** 2)
            else:
                res = o.Z[l][V[m]] - pre
                total += np.sum(o.U[V[m]] * res) + 0.5 * o.p.rho * np.sum(res ** 2)
        assert abs(total - o.phi(l, o.W[l])) <= 1e-12 * max(1.0, abs(total))
    # propagation row for row
    for m in range(o.M):
        split = sum(At[np.ix_(V[m], V[r])] @ o.Z[1][V[r]] for r in range(o.M))
        np.testing.assert_allclose(split, (o.At @ o.Z[1])[V[m]], atol=1e-13)


@pytest.mark.parametrize("seed", [0, 1, 4])
def test_gradients_by_finite_differences(seed):
    pr, o = make(seed, n=14, widths=(4, 5, 3, 3))
    assert keep_off_kinks(o, 1e-4)
    for l in range(1, o.L + 1):
        g = o.grad_phi(l)
        gn = num_grad(lambda w: o.phi(l, w), o.W[l])
        np.testing.assert_allclose(g, gn, rtol=2e-6, atol=2e-7)
    for l in range(1, o.L):
        for m in range(o.M):
            g = o.grad_psi(l, m)
            gn = num_grad(lambda z: psi_message_form(pr, o, l, m, z), o.Z[l][o.V[m]])
            np.testing.assert_allclose(g, gn, rtol=2e-6, atol=2e-7)
    # output layer rows
    L = o.L
    q = (o.At @ o.Z[L - 1]) @ o.W[L]
    rows = np.arange(o.n)
    g = o.grad_psi_L_rows(o.Z[L], q, o.U, o.y)
    for i in np.flatnonzero(o.train)[:4]:
        f = lambda z: o.psi_L_rows(z[None], q[i:i + 1], o.U[i:i + 1], o.y[i:i + 1], np.array([True]))[0]
        np.testing.assert_allclose(g[i], num_grad(f, o.Z[L][i]), rtol=2e-6, atol=2e-7)


@pytest.mark.parametrize("seed", [0, 2])
def test_community_gradient_is_rows_of_full_gradient(seed):
    pr, o = make(seed)
    At = dense_At(pr)
    nu, rho, L = o.p.nu, o.p.rho, o.L
    for l in range(1, L):
        H = At @ o.Z[l - 1] @ o.W[l]
        Hn = At @ o.Z[l] @ o.W[l + 1]
        if l + 1 < L:
            back = nu * (np.maximum(Hn, 0) - o.Z[l + 1]) * (Hn > 0)
        else:
            back = -(o.U + rho * (o.Z[L] - Hn))
        full = nu * (o.Z[l] - np.maximum(H, 0)) + At.T @ back @ o.W[l + 1].T
        for m in range(o.M):
            np.testing.assert_allclose(o.grad_psi(l, m), full[o.V[m]], atol=1e-12)
    # and the partition does not matter for the gradient
    pr1 = dict(pr, community=np.zeros(pr["n"], dtype=np.int64), n_comm=1)
    o1 = orc.OracleADMM(pr1["n"], pr1["row_ptr"], pr1["col_idx"], pr1["X"], pr1["y"], pr1["mask"],
                        pr1["widths"], o.p, 1, pr1["community"], pr1["W"])
    o1.Z, o1.U = o.Z, o.U
    np.testing.assert_allclose(o1.grad_psi(1, 0), full_gradient_layer1(At, o), atol=1e-12)


def full_gradient_layer1(At, o):
    nu, rho, L = o.p.nu, o.p.rho, o.L
    H = At @ o.Z[0] @ o.W[1]
    Hn = At @ o.Z[1] @ o.W[2]
    back = nu * (np.maximum(Hn, 0) - o.Z[2]) * (Hn > 0) if 2 < L else -(o.U + rho * (o.Z[L] - Hn))
    return nu * (o.Z[1] - np.maximum(H, 0)) + At.T @ back @ o.W[2].T


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_search_condition_and_monotone_blocks(seed):
    pr, o = make(seed)
    for l in range(1, o.L + 1):
        o.tau[l] = 1e-3                      # start low so that several trials are rejected
        Wn, t, rec = o.update_W(l)
        assert rec["trial"] >= 1
        f0, f1 = o.phi(l, o.W[l]), o.phi(l, Wn)
        g = o.grad_phi(l)
        gg = np.sum(g * g)
        assert f1 <= f0 - gg / (2 * t) + 1e-15 * abs(f0)
        assert f1 <= f0
        np.testing.assert_allclose(Wn, o.W[l] - g / t, atol=0, rtol=1e-15)
        t_before = t / o.p.bt_growth          # the previous trial must have failed
        assert o.phi(l, o.W[l] - g / t_before) > f0 - gg / (2 * t_before)
        assert abs(t - 1e-3 * o.p.bt_shrink * o.p.bt_growth ** rec["trial"]) <= 1e-12 * t
    for l in range(1, o.L):
        for m in range(o.M):
            o.theta[l][m] = 1e-3
            Zn, t, rec = o.update_Z(l, m, o.W)
            g = o.grad_psi(l, m)
            gg = np.sum(g * g)
            f0, f1 = o.psi(l, m, o.Z[l][o.V[m]]), o.psi(l, m, Zn)
            assert f1 <= f0 - gg / (2 * t) + 1e-15 * abs(f0)
            if rec["trial"] >= 1:
                tb = t / o.p.bt_growth
                assert o.psi(l, m, o.Z[l][o.V[m]] - g / tb) > f0 - gg / (2 * tb)
            np.testing.assert_allclose(Zn, o.Z[l][o.V[m]] - g / t, rtol=1e-15)


@pytest.mark.parametrize("seed", [0, 5])
def test_last_layer_W_block_is_quadratic(seed):
    """phi_L is exactly quadratic in W_L with Hessian rho * P^T P (Kronecker identity), so every
    tau >= rho * lambda_max passes and doubling cannot overshoot 2 * max(start, rho*lambda_max)."""
    pr, o = make(seed)
    L = o.L
    P = dense_At(pr) @ o.Z[L - 1]
    lam = o.p.rho * np.linalg.eigvalsh(P.T @ P).max()
    g = o.grad_phi(L)
    gg = np.sum(g * g)
    f0 = o.phi(L, o.W[L])
    for t in (lam, 1.7 * lam, 10 * lam):
        assert o.phi(L, o.W[L] - g / t) <= f0 - gg / (2 * t) + 1e-12 * abs(f0)
    for start in (1e-4, 3.0 * lam):
        o.tau[L] = start / o.p.bt_shrink
        _, t, rec = o.update_W(L)
        assert t < 2 * max(start, lam) * (1 + 1e-12)


def test_first_iteration_from_consistent_start_moves_only_ZL():
    pr, o = make(7, perturb=0)
    W0 = [None] + [w.copy() for w in o.W[1:]]
    Z0 = [z.copy() for z in o.Z]
    rec = o.iterate()
    for l in range(1, o.L + 1):
        np.testing.assert_array_equal(o.W[l], W0[l])
        assert rec["W"][l]["trial"] == orc.SKIPPED
    for l in range(1, o.L):
        np.testing.assert_array_equal(o.Z[l], Z0[l])
    np.testing.assert_array_equal(o.U, np.zeros_like(o.U))
    assert np.abs(o.Z[o.L] - Z0[o.L])[o.train].max() > 1e-3
    np.testing.assert_allclose(o.Z[o.L][~o.train], Z0[o.L][~o.train], atol=1e-13)


def test_output_layer_rows():
    pr, o = make(9)
    L, rho, s = o.L, o.p.rho, o.p.loss_scale
    q = dense_At(pr) @ o.Z[L - 1] @ o.W[L]
    Zn = o.update_ZL(o.W, iters=6000)
    off = ~o.train
    np.testing.assert_allclose(Zn[off], q[off] - o.U[off] / rho, atol=1e-13)   # closed form
    # training rows: stationarity, and agreement with Newton's method on the same objective
    for i in np.flatnonzero(o.train):
        z = Zn[i]
        sm = np.exp(z - z.max()); sm /= sm.sum()
        e = np.zeros_like(z); e[o.y[i]] = 1
        assert np.abs(s * (sm - e) + o.U[i] + rho * (z - q[i])).max() < 1e-9
        x = o.Z[L][i].copy()
        for _ in range(100):
            sm = np.exp(x - x.max()); sm /= sm.sum()
            grad = s * (sm - e) + o.U[i] + rho * (x - q[i])
            hess = s * (np.diag(sm) - np.outer(sm, sm)) + rho * np.eye(len(x))
            x = x - np.linalg.solve(hess, grad)
        np.testing.assert_allclose(z, x, atol=1e-8)
    # the default iteration count is a truncation of the same sequence: it must lower the objective
    Z30 = o.update_ZL(o.W)
    tr = o.train
    before = o.psi_L_rows(o.Z[L], q, o.U, o.y, tr).sum()
    assert o.psi_L_rows(Z30, q, o.U, o.y, tr).sum() < before


def test_fista_matches_textbook_sequence_on_one_row():
    """The momentum sequence t_{j+1} = (1 + sqrt(1 + 4 t_j^2)) / 2 and the extrapolation
    y_{j+1} = x_j + (t_j - 1)/t_{j+1} (x_j - x_{j-1}), checked by a scalar re-run."""
    pr, o = make(11)
    L, p = o.L, o.p
    i = int(np.flatnonzero(o.train)[0])
    q = (dense_At(pr) @ o.Z[L - 1] @ o.W[L])[i]
    u, yi = o.U[i], o.y[i]
    x_prev = o.Z[L][i].copy(); v = x_prev.copy(); t = 1.0
    step = 1.0 / (0.5 * p.loss_scale + p.rho)
    ts = [1.0]
    for _ in range(p.fista_iters):
        sm = np.exp(v - v.max()); sm /= sm.sum(); sm[yi] -= 1
        x = v - step * (p.loss_scale * sm + u + p.rho * (v - q))
        tn = (1 + np.sqrt(1 + 4 * t * t)) / 2
        v = x + (t - 1) / tn * (x - x_prev)
        x_prev, t = x, tn
        ts.append(t)
    assert abs(ts[1] - (1 + np.sqrt(5)) / 2) < 1e-15 and ts[2] > ts[1]
    np.testing.assert_allclose(o.update_ZL(o.W)[i], x_prev, atol=1e-13)


def test_dual_update_closed_form_both_modes():
    pr, o = make(13)
    At = dense_At(pr)
    L = o.L
    for mode in (0, 1):
        pr2, o2 = make(13)
        o2.p.dual_mode = mode
        Zk, Uk = [z.copy() for z in o2.Z], o2.U.copy()
        o2.iterate()
        Zuse = Zk if mode == 0 else o2.Z
        expect = Uk + o2.p.rho * (Zuse[L] - At @ Zuse[L - 1] @ o2.W[L])
        np.testing.assert_allclose(o2.U, expect, atol=1e-13)


def test_objective_and_predict():
    pr, o = make(17, perturb=0)
    obj = o.objective()
    assert abs(obj[0] - obj[1]) < 1e-12 and abs(obj[2]) < 1e-20 and abs(obj[4]) < 1e-20
    At = dense_At(pr)
    Z = pr["X"]
    for l in range(1, o.L + 1):
        Z = At @ Z @ pr["W"][l - 1]
        if l < o.L:
            Z = np.maximum(Z, 0)
    logits, labels = o.predict()
    np.testing.assert_allclose(logits, Z, atol=1e-12)
    assert labels.tolist() == [int(np.argmax(r)) for r in Z]
    tr = np.flatnonzero(o.train)
    ce = -np.log(np.exp(Z[tr, o.y[tr]]) / np.exp(Z[tr]).sum(axis=1)).sum()
    assert abs(obj[1] - ce) < 1e-10
    assert abs(obj[5] - np.mean(np.argmax(Z[tr], 1) == o.y[tr])) < 1e-15
    # after a perturbation every term is active and L_rho is their sum
    pr, o = make(17)
    obj = o.objective()
    r = o.Z[o.L] - At @ o.Z[o.L - 1] @ o.W[o.L]
    assert abs(obj[3] - np.sum(o.U * r)) < 1e-12 and abs(obj[4] - 0.5 * o.p.rho * np.sum(r * r)) < 1e-12
    assert abs(obj[0] - obj[1:5].sum()) < 1e-12 and obj[2] > 0


def test_components_as_communities_run_independently():
    """When every community is a union of connected components there is no cross edge; the Z
    blocks of the M-community run then equal those of separate single-community problems
    that share the same W (the W block is global, so it is compared on the joint problem)."""
    rng = np.random.default_rng(21)
    n1, n2 = 10, 13
    from conftest import random_graph
    _, _, A1 = random_graph(rng, n1, 0.4)
    _, _, A2 = random_graph(rng, n2, 0.35)
    A = np.zeros((n1 + n2, n1 + n2)); A[:n1, :n1] = A1; A[n1:, n1:] = A2
    from conftest import dense_to_csr
    widths = [4, 5, 3]
    X = rng.standard_normal((n1 + n2, 4)); y = rng.integers(0, 3, n1 + n2)
    mask = (rng.random(n1 + n2) < 0.4).astype(np.uint8)
    W = [0.5 * rng.standard_normal((4, 5)), 0.5 * rng.standard_normal((5, 3))]
    comm = np.array([0] * n1 + [1] * n2)
    params = orc.Params(nu=0.5, rho=0.8)
    o = orc.OracleADMM(n1 + n2, *dense_to_csr(A), X, y, mask, widths, params, 2, comm, W)
    assert all(len(x) == 0 for x in o.nbr)
    dZ = 0.3 * rng.standard_normal(o.Z[1].shape)
    o.Z[1] = o.Z[1] + dZ
    o.U = 0.3 * rng.standard_normal(o.U.shape)
    parts = []
    for sl, Asub in ((slice(0, n1), A1), (slice(n1, None), A2)):
        k = Asub.shape[0]
        s = orc.OracleADMM(k, *dense_to_csr(Asub), X[sl], y[sl], mask[sl], widths, params, 1,
                           np.zeros(k, dtype=int), W)
        s.Z[1] = o.Z[1][sl].copy(); s.Z[2] = o.Z[2][sl].copy(); s.U = o.U[sl].copy()
        parts.append(s)
    for m, s in enumerate(parts):
        Zn, t, rec = o.update_Z(1, m, o.W)
        Zs, ts, recs = s.update_Z(1, 0, s.W)
        np.testing.assert_allclose(Zn, Zs, atol=1e-13)
        assert rec["trial"] == recs["trial"] and abs(t - ts) < 1e-15


def test_replay_mode_reproduces_free_run():
    pr, o = make(23)
    pr, o2 = make(23)
    recs = [o.iterate() for _ in range(3)]
    for rec in recs:
        forced = dict(W={l: r["trial"] for l, r in rec["W"].items()},
                      Z={k: r["trial"] for k, r in rec["Z"].items()})
        rec2 = o2.iterate(forced)
        assert all(r["ok"] for r in rec2["W"].values()) and all(r["ok"] for r in rec2["Z"].values())
    for l in range(1, o.L + 1):
        np.testing.assert_array_equal(o.W[l], o2.W[l])
        np.testing.assert_array_equal(o.Z[l], o2.Z[l])
    np.testing.assert_array_equal(o.U, o2.U)


def test_large_nu_pulls_hidden_layers_to_the_network():
    """nu -> infinity turns the relaxed problem back into the constrained one (Problem 2 text):
    with a large nu the Z_1 step moves Z_1 towards f_1(A~ Z_0 W_1)."""
    pr, o = make(29, nu=1e4, rho=1e-3)
    target = np.maximum((o.At @ o.Z[0]) @ o.W[1], 0)
    before = np.linalg.norm(o.Z[1] - target)
    for _ in range(5):
        o.iterate()
    target = np.maximum((o.At @ o.Z[0]) @ o.W[1], 0)
    assert np.linalg.norm(o.Z[1] - target) < 0.5 * before


def test_sampled_row_evaluator_matches_the_full_oracle():
    """oracle/sampled_rows.py (used where a full pass is out of reach) against the full oracle."""
    from oracle.sampled_rows import SampledRows
    pr, o = make(31)
    sr = SampledRows(pr["n"], pr["row_ptr"], pr["col_idx"], pr["y"], pr["mask"], pr["widths"], o.p.nu, o.p.rho)
    rows = np.arange(pr["n"])
    At = dense_At(pr)
    np.testing.assert_allclose(sr.propagate_rows(o.Z[1], rows), At @ o.Z[1], atol=1e-13)
    for l in range(1, o.L + 1):
        np.testing.assert_allclose(sr.H_rows(l, rows, o.Z, o.W), At @ o.Z[l - 1] @ o.W[l], atol=1e-12)
    for l in range(1, o.L):
        full = np.zeros_like(o.Z[l])
        for m in range(o.M):
            full[o.V[m]] = o.grad_psi(l, m)
        np.testing.assert_allclose(sr.grad_Z_rows(l, rows, o.Z, o.W, o.U), full, atol=1e-12)
    np.testing.assert_allclose(sr.ZL_rows(rows, o.Z, o.W, o.U), o.update_ZL(o.W), atol=1e-12)
    np.testing.assert_allclose(sr.U_rows(rows, o.Z, o.W, o.U), o.update_U(o.W, o.Z), atol=1e-13)
    np.testing.assert_allclose(sr.adj_rows(rows[::3]).toarray(), At[::3], atol=1e-15)


@pytest.mark.parametrize("seed,widths", [(33, (5, 6, 4, 3)), (34, (4, 5, 3)), (35, (3, 4, 4, 5, 2))])
def test_community_step_condition_evaluator_matches_psi(seed, widths):
    """``SampledRows.psi_change`` (objective change of one community along its step, from the community's
    rows and their neighbours only) against differences of the full oracle's literal psi_m, and its
    ||grad||^2 against grad_psi; the accepted theta of the oracle's own search must pass by it and the
    trial before must fail."""
    from oracle.sampled_rows import SampledRows
    pr, o = make(seed, n=30, widths=widths, n_comm=4)
    sr = SampledRows(pr["n"], pr["row_ptr"], pr["col_idx"], pr["y"], pr["mask"], pr["widths"], o.p.nu, o.p.rho)
    for l in range(1, o.L):
        for m in range(o.M):
            g = o.grad_psi(l, m)
            thetas = [0.05, 0.4, 3.0, 50.0]
            gg, change = sr.psi_change(l, o.V[m], o.Z, o.W, o.U, thetas)
            assert abs(gg - np.sum(g * g)) <= 1e-12 * max(gg, 1e-300)
            f0 = o.psi(l, m, o.Z[l][o.V[m]])
            for t, c in zip(thetas, change):
                want = o.psi(l, m, o.Z[l][o.V[m]] - g / t) - f0
                assert abs(c - want) <= 1e-11 * max(abs(f0), 1.0), (l, m, t, c, want)
            o.theta[l][m] = 1e-3
            _, t, rec = o.update_Z(l, m, o.W)
            assert rec["trial"] >= 1
            gg, (c_acc, c_prev) = sr.psi_change(l, o.V[m], o.Z, o.W, o.U, [t, t / o.p.bt_growth])
            assert -c_acc >= gg / (2 * t) and -c_prev < gg / (2 * (t / o.p.bt_growth))
            assert abs(-c_acc / (gg / (2 * t)) - rec["q"]) <= 1e-9 * abs(rec["q"])


@pytest.mark.parametrize("seed,n_comm", [(41, 1), (42, 3)])
def test_sequential_schedule_descends_block_by_block(seed, n_comm):
    """In the serial schedule every accepted W / hidden-Z step is a majorisation step on the augmented
    Lagrangian as a function of that block with all other blocks at their latest values, so L_rho of Eq. 1
    cannot go up across such a block (with one community; with several, the communities of a layer move
    together from the same point and the bound holds per community objective, so a small slack is allowed).
    A schedule that read stale values would not have this property."""
    pr, o = make(seed, n_comm=n_comm)
    prev = o.objective()[0]
    for it in range(3):
        trace = []
        o.iterate_sequential(trace=trace)
        for kind, l, val in trace:
            hidden_or_w = kind == "W" or l < o.L
            slack = (1e-12 if n_comm == 1 else 5e-3) * max(1.0, abs(prev))
            if hidden_or_w:
                assert val <= prev + slack, (it, kind, l, prev, val)
            prev = val
        prev = o.objective()[0]       # after the dual step


def test_sequential_schedule_uses_latest_values():
    """One pass by hand: W_1 from the old state, Z_1 with the new W_1 and the old W_2, W_2 with the new Z_1."""
    pr, o = make(43)
    pr, ref = make(43)
    o.iterate_sequential()
    W1, t, _ = ref.update_W(1)
    ref.W[1], ref.tau[1] = W1, t
    Z1 = ref.Z[1].copy()
    for m in range(ref.M):
        Z1[ref.V[m]], ref.theta[1][m], _ = ref.update_Z(1, m, ref.W)
    ref.Z[1] = Z1
    W2, t, _ = ref.update_W(2)
    np.testing.assert_array_equal(o.W[1], W1)
    np.testing.assert_array_equal(o.Z[1], Z1)
    np.testing.assert_array_equal(o.W[2], W2)


# ---- time indices of Algorithm 1 (Appendix A, first display; Eq. 3) -------------------------

def dense_hidden_gradient(At, nu, rho, L, l, W, Z, U):
    """Full-graph gradient of the Z_l objective (Eq. 5 / Eq. 6) from dense matrices, with the
    weights, states and dual handed in, so the caller chooses the time index of each."""
    H = At @ Z[l - 1] @ W[l]
    Hn = At @ Z[l] @ W[l + 1]
    if l + 1 < L:
        back = nu * (np.maximum(Hn, 0) - Z[l + 1]) * (Hn > 0)
    else:
        back = -(U + rho * (Z[L] - Hn))
    return nu * (Z[l] - np.maximum(H, 0)) + At.T @ back @ W[l + 1].T


@pytest.mark.parametrize("seed,dual_mode", [(51, 0), (52, 1), (53, 0)])
def test_one_pass_reads_the_iterates_algorithm_1_names(seed, dual_mode):
    """Algorithm 1 with Appendix A's first display: every W_l from (W^k, Z^k, U^k); every Z_{l,m} and Z_L
    from (W^{k+1}, Z^k, U^k), layers and communities in parallel; U by Eq. 3.  Checked two ways:
    against dense-matrix formulas evaluated at those iterates (the step times its parameter must be
    the gradient there), and against a pass assembled by hand from single block updates of a twin."""
    pr, o = make(seed, n=26, widths=(5, 6, 4, 4, 3))
    pr, ref = make(seed, n=26, widths=(5, 6, 4, 4, 3))
    o.p.dual_mode = ref.p.dual_mode = dual_mode
    for x in (o, ref):                       # low starting parameters: every search runs a few trials
        x.tau = [None] + [1e-2] * x.L
        x.theta = [None] + [[1e-2] * x.M for _ in range(1, x.L)]
    At = dense_At(pr)
    L, M, nu, rho = o.L, o.M, o.p.nu, o.p.rho
    Wk = [None] + [w.copy() for w in o.W[1:]]
    Zk = [z.copy() for z in o.Z]
    Uk = o.U.copy()
    rec = o.iterate()
    assert all(r["trial"] >= 0 for r in rec["W"].values()) and all(r["trial"] >= 0 for r in rec["Z"].values())

    # (a) dense formulas at the iterates the paper names
    for l in range(1, L + 1):
        P = At @ Zk[l - 1]
        H = P @ Wk[l]
        if l < L:
            g = nu * P.T @ ((np.maximum(H, 0) - Zk[l]) * (H > 0))
        else:
            g = -P.T @ (Uk + rho * (Zk[L] - H))
        np.testing.assert_allclose((Wk[l] - o.W[l]) * o.tau[l], g, rtol=1e-9, atol=1e-12)
    for l in range(1, L):
        G = dense_hidden_gradient(At, nu, rho, L, l, o.W, Zk, Uk)        # W^{k+1}, Z^k, U^k
        for m in range(M):
            Vm = o.V[m]
            np.testing.assert_allclose((Zk[l][Vm] - o.Z[l][Vm]) * o.theta[l][m], G[Vm], rtol=1e-9, atol=1e-12)
        # the neighbouring readings (W^k; layers below l already at k+1) give a different matrix
        assert np.abs(dense_hidden_gradient(At, nu, rho, L, l, Wk, Zk, Uk) - G).max() > 1e-6
        if l > 1:
            Zgs = [o.Z[j] if 1 <= j < l else Zk[j] for j in range(L + 1)]
            assert np.abs(dense_hidden_gradient(At, nu, rho, L, l, o.W, Zgs, Uk) - G).max() > 1e-6
    off = ~o.train
    q = At @ Zk[L - 1] @ o.W[L]                                           # Z_{L-1}^k with W_L^{k+1}
    np.testing.assert_allclose(o.Z[L][off], q[off] - Uk[off] / rho, atol=1e-11)
    assert np.abs(q - At @ Zk[L - 1] @ Wk[L]).max() > 1e-6 and np.abs(q - At @ o.Z[L - 1] @ o.W[L]).max() > 1e-6
    Zd = Zk if dual_mode == 0 else o.Z
    np.testing.assert_allclose(o.U, Uk + rho * (Zd[L] - At @ Zd[L - 1] @ o.W[L]), atol=1e-12)

    # (b) the same pass assembled from single block updates of the twin
    Wn, taun = list(ref.W), list(ref.tau)
    for l in range(1, L + 1):
        Wn[l], taun[l], _ = ref.update_W(l)
    Zn = [z.copy() for z in ref.Z]
    thetan = [None] + [list(t) for t in ref.theta[1:]]
    for l in range(1, L):
        for m in range(M):
            Zn[l][ref.V[m]], thetan[l][m], _ = ref.update_Z(l, m, Wn)      # ref.Z, ref.U still at k
    Zn[L] = ref.update_ZL(Wn)
    Un = ref.update_U(Wn, ref.Z if dual_mode == 0 else Zn)
    for l in range(1, L + 1):
        np.testing.assert_array_equal(o.W[l], Wn[l])
        np.testing.assert_array_equal(o.Z[l], Zn[l])
        assert o.tau[l] == taun[l]
    for l in range(1, L):
        assert o.theta[l] == thetan[l]
    np.testing.assert_array_equal(o.U, Un)


def test_train_accuracy_is_that_of_the_forward_pass():
    """Entry 5 of objective() is the accuracy of predict() (Problem 1's network with the current W), not
    of the auxiliary Z_L: away from the forward-consistent start the two differ."""
    pr, o = make(57, n=40, n_train=30, perturb=0)
    rng = np.random.default_rng(5)
    o.Z[o.L] = rng.standard_normal(o.Z[o.L].shape) * 3.0       # Z_L no longer the network's output
    At = dense_At(pr)
    Z = pr["X"]
    for l in range(1, o.L + 1):
        Z = At @ Z @ o.W[l]
        if l < o.L:
            Z = np.maximum(Z, 0)
    tr = np.flatnonzero(o.train)
    acc_net = np.mean(np.argmax(Z[tr], 1) == o.y[tr])
    acc_aux = np.mean(np.argmax(o.Z[o.L][tr], 1) == o.y[tr])
    assert acc_net != acc_aux
    assert o.objective()[5] == acc_net
