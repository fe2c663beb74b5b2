"""Degenerate and ragged inputs through the C ABI, against the oracle: one community, no edges
at all, a single layer, all / no training rows, widths that are not multiples of four."""
import numpy as np
import pytest

from conftest import tiny_problem
from oracle import gcn_admm_oracle as orc
from paper_2112_09335_b200 import binding
from parity_utils import relerr

pytestmark = pytest.mark.gpu


def run_pair(pr, n_it=4, **params):
    kw = dict(nu=0.05, rho=0.08)
    kw.update(params)
    w32 = [w.astype(np.float32) for w in pr["W"]]
    g = binding.GcnAdmm(pr["n"], pr["row_ptr"], pr["col_idx"], pr["X"].astype(np.float32), pr["y"], pr["mask"],
                        pr["widths"], pr["n_comm"], pr["community"], w32, **kw)
    o = orc.OracleADMM(pr["n"], pr["row_ptr"], pr["col_idx"], pr["X"].astype(np.float32), pr["y"], pr["mask"],
                       pr["widths"], orc.Params(**kw), pr["n_comm"], pr["community"], w32)
    try:
        g.step(n_it)
        dec = g.decisions()
        for k in range(n_it):
            L, M = o.L, o.M
            forced = dict(W={l: int(dec["trial_w"][k, l - 1]) for l in range(1, L + 1)},
                          Z={(l, m): int(dec["trial_z"][k, l - 1, m]) for l in range(1, L) for m in range(M)})
            o.forced_tol = 1e-4
            rec = o.iterate(forced)
            assert all(r["ok"] for r in list(rec["W"].values()) + list(rec["Z"].values())), (k, rec)
        for l in range(1, o.L + 1):
            assert relerr(g.get_state(binding.ST_W, l), o.W[l]) < 1e-4
            assert relerr(g.get_state(binding.ST_Z, l), o.Z[l]) < 1e-4
        assert relerr(g.get_state(binding.ST_U), o.U) < 1e-4
        go, oo = g.objective(), o.objective()
        assert abs(go[0] - oo[0]) <= 1e-4 * np.abs(oo[1:5]).sum()
    finally:
        g.destroy()


def test_single_community():
    run_pair(tiny_problem(1, n=70, widths=(9, 13, 5), n_comm=1))


def test_three_layers_odd_widths():
    run_pair(tiny_problem(2, n=90, widths=(11, 7, 10, 3), n_comm=5))


def test_graph_without_edges_is_an_mlp():
    pr = tiny_problem(3, n=40, widths=(6, 8, 4), n_comm=3, p=0.0)
    assert pr["col_idx"].size == 0
    run_pair(pr)


def test_single_layer():
    run_pair(tiny_problem(4, n=50, widths=(8, 4), n_comm=2))


def test_all_rows_training_and_none():
    pr = tiny_problem(5, n=60, widths=(5, 6, 3), n_comm=4)
    pr["mask"][:] = 1
    run_pair(pr)
    pr["mask"][:] = 0
    run_pair(pr)


def test_many_small_communities_and_isolated_nodes():
    pr = tiny_problem(6, n=120, widths=(7, 12, 6), n_comm=40, p=0.03)
    run_pair(pr)


def test_dual_mode_one_and_other_search_parameters():
    pr = tiny_problem(7, n=80, widths=(6, 9, 4), n_comm=3)
    run_pair(pr, dual_mode=1, bt_growth=3.0, bt_shrink=0.3, tau0=0.01, theta0=0.02, fista_iters=7, loss_scale=0.5)


def test_first_hidden_layer_wider_than_1024():
    """Only C_2 .. C_L are limited to 1024 columns (the row width of the theta scoring); C_0 and C_1 may be
    wider.  A three-layer net with C_1 = 1100 must run and match; C_2 = 1100 must be refused."""
    run_pair(tiny_problem(8, n=48, widths=(6, 1100, 5, 3), n_comm=3), n_it=3)
    pr = tiny_problem(8, n=48, widths=(6, 7, 1100, 3), n_comm=3)
    with pytest.raises(binding.GcnAdmmError) as e:
        binding.GcnAdmm(pr["n"], pr["row_ptr"], pr["col_idx"], pr["X"].astype(np.float32), pr["y"], pr["mask"],
                        pr["widths"], pr["n_comm"], pr["community"], [w.astype(np.float32) for w in pr["W"]])
    assert e.value.code == -4


@pytest.mark.parametrize("n,widths,n_comm", [(2000, (6, 9, 7, 4), 400), (2400, (6, 8, 4), 800)])
def test_more_communities_than_shared_memory_holds(n, widths, n_comm):
    """The theta scoring keeps its per-community sums in shared memory while they fit (384 communities with
    four candidates, 768 with the closed form); beyond that a warp adds into its chunk's slice in global
    memory.  400 communities put the hidden-layer scoring on that path, 800 the output-layer scoring too."""
    pr = tiny_problem(9, n=n, widths=widths, n_comm=n_comm, p=4.0 / n)
    run_pair(pr, n_it=3)
