"""The largest workload at full size (2.45 M nodes, ~62 M edges, 100-256-256-47, 64 communities), in the
launch configuration bench.py times.  A full oracle pass is out of reach there, so sampled outputs are
checked against rows the fp64 oracle computes one by one (oracle/sampled_rows.py): propagation rows, the
hidden Z block updates (given the accepted theta, whose decision is logged), the output-layer rows and
the dual rows; the step-size decision of sampled communities is re-evaluated in fp64 from the community's
rows and their neighbours (the accepted trial must satisfy the condition of Eq. 9, the one before it must
not); plus properties that hold at any size (no exhausted search, every accepted q >= 1)."""
import numpy as np
import pytest

from oracle.sampled_rows import SampledRows
from paper_2112_09335_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def rows_close(got, want, scale, tol):
    err = np.abs(np.asarray(got, dtype=np.float64) - want)
    return float(np.max(err / (scale + 1e-30))), tol


@pytest.fixture(scope="module")
def wl_full():
    return inputs.make_workload(4)


def test_two_runs_give_the_same_bits_at_full_size(wl_full):
    """At this size the chunks of the theta scoring are taken by whichever warp is free, thousands at a time;
    the sums are kept per chunk and added in chunk order, so two runs must still agree bit for bit."""
    wl = wl_full
    L = len(wl.widths) - 1
    outs = []
    for _ in range(2):
        g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                            wl.w_init, nu=wl.nu, rho=wl.rho)
        try:
            g.step(6)
            d = g.decisions()
            outs.append(dict(trial_w=d["trial_w"], trial_z=d["trial_z"], q_w=d["q_w"], q_z=d["q_z"], obj=g.objective(),
                             ZL=g.get_state(binding.ST_Z, L), U=g.get_state(binding.ST_U),
                             **{f"W{l}": g.get_state(binding.ST_W, l) for l in range(1, L + 1)},
                             **{f"theta{l}": g.get_state(binding.ST_THETA, l) for l in range(1, L)}))
        finally:
            g.destroy()
    assert (outs[0]["trial_z"][3:] >= 0).all()          # the searches were really running
    for key in outs[0]:
        assert np.array_equal(outs[0][key], outs[1][key]), key


def test_sampled_rows_at_full_size(wl_full):
    import torch
    wl = wl_full
    g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                        wl.w_init, nu=wl.nu, rho=wl.rho)
    try:
        L, M = len(wl.widths) - 1, wl.n_comm
        sr = SampledRows(wl.n, wl.row_ptr, wl.col_idx, wl.y, wl.train_mask, wl.widths, wl.nu, wl.rho)
        rng = np.random.default_rng(5)
        deg = np.diff(wl.row_ptr)
        train_rows = np.flatnonzero(wl.train_mask)
        rows = np.unique(np.concatenate([rng.choice(wl.n, 12, replace=False), rng.choice(train_rows, 4, replace=False),
                                         [int(np.argmax(deg)), int(np.argmin(deg))]]))
        # ---- propagation rows ----
        x = torch.randn(wl.n, 32, device="cuda", generator=torch.Generator(device="cuda").manual_seed(1))
        out = torch.empty_like(x)
        g.propagate(x.data_ptr(), 32, out=out.data_ptr())
        torch.cuda.synchronize()
        xh = x.cpu().numpy()
        want = sr.propagate_rows(xh, rows)
        mag = np.zeros_like(want)
        for k, i in enumerate(rows):
            c, v = sr.adj_row(int(i))
            mag[k] = v @ np.abs(xh[c])
        worst, _ = rows_close(out[torch.from_numpy(rows).cuda()].cpu().numpy(), want, mag, 0)
        assert worst < 2e-6, worst
        del x, out, xh

        # ---- a state with every term active: three passes from the forward start ----
        g.step(3)
        dec = g.decisions()
        assert (dec["trial_w"] != -2).all() and (dec["trial_z"] != -2).all()
        ok = dec["trial_w"] >= 0
        assert (dec["q_w"][ok] >= 1.0).all()
        okz = dec["trial_z"] >= 0
        assert (dec["q_z"][okz] >= 1.0).all()

        def fetch():
            Z = [wl.X] + [g.get_state(binding.ST_Z, l) for l in range(1, L + 1)]
            W = [None] + [g.get_state(binding.ST_W, l) for l in range(1, L + 1)]
            return Z, W, g.get_state(binding.ST_U)

        report = {}
        for l in range(1, L):                      # hidden Z blocks: Z_new = Z - grad / theta_{comm(row)}
            Z, W, U = fetch()
            # start every search of this layer three doublings lower, so that accepted trials are preceded
            # by rejected ones and both sides of the condition can be checked
            g.set_state(binding.ST_THETA, l, g.get_state(binding.ST_THETA, l) / 8.0)
            g.step_block(binding.PHASE_Z, l)
            theta = g.get_state(binding.ST_THETA, l)
            dz = g.decisions()
            trial, q_gpu = dz["trial_z"][0, l - 1], dz["q_z"][0, l - 1]
            assert (trial >= 0).all()
            # Eq. 9 in fp64 for two communities: the one whose decision was tightest, and a random other one
            tight = int(np.argmin(np.abs(q_gpu - 1.0)))
            for m in (tight, int((tight + 1 + rng.integers(0, M - 1)) % M)):
                t_acc = float(theta[m])
                gg, (c_acc, c_prev) = sr.psi_change(l, np.flatnonzero(wl.community == m), Z, W, U, [t_acc, t_acc / 2.0])
                q_acc, q_prev = -c_acc / (gg / (2.0 * t_acc)), -c_prev / (gg / t_acc)
                report[f"theta{l},{m}"] = (q_acc, q_gpu[m])
                assert q_acc >= 1.0 - 1e-4, (l, m, q_acc)
                assert trial[m] == 0 or q_prev < 1.0 + 1e-4, (l, m, trial[m], q_prev)
                assert abs(q_gpu[m] - q_acc) <= 2e-3 * abs(q_acc), (l, m, q_gpu[m], q_acc)
            got = g.get_state(binding.ST_Z, l)[rows]
            grad = sr.grad_Z_rows(l, rows, Z, W, U)
            comm = wl.community[rows]
            stepped = trial[comm] >= 0
            want = Z[l][rows].astype(np.float64) - np.where(stepped[:, None], grad / theta[comm][:, None], 0.0)
            assert stepped.any()
            rel = np.linalg.norm(got - want) / np.linalg.norm(want)
            rel_step = np.linalg.norm((got - Z[l][rows]) - (want - Z[l][rows])) / max(np.linalg.norm(want - Z[l][rows]), 1e-300)
            report[f"Z{l}"] = (rel, rel_step)
            assert rel < 1e-5 and rel_step < 5e-3, (l, rel, rel_step)
        Z, W, U = fetch()                            # output layer rows, Eq. (7)
        g.step_block(binding.PHASE_Z, L)
        got = g.get_state(binding.ST_Z, L)[rows]
        want = sr.ZL_rows(rows, Z, W, U)
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        report[f"Z{L}"] = (rel, 0.0)
        assert rel < 1e-5, rel
        Z, W, U = fetch()                            # dual rows, Eq. (3)
        g.step_block(binding.PHASE_U, 0)
        got = g.get_state(binding.ST_U)[rows]
        want = sr.U_rows(rows, Z, W, U)
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        report["U"] = (rel, 0.0)
        assert rel < 1e-5, rel
        print("\n  full size, sampled rows:", {k: (f"{a:.1e}", f"{b:.1e}") for k, (a, b) in report.items()})
    finally:
        g.destroy()
