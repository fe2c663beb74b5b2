"""Two runs from the same inputs give the same bits.  Every sum that decides a step size is formed in a fixed
order (per-block partial sums, added up by one block or one warp in index order), so the weights, the
auxiliary variables, the dual, the step parameters, the accepted trials and the reported objective of two
handles built from the same inputs must be identical, not merely close."""
import numpy as np
import pytest

from paper_2112_09335_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def run(wl, passes, **kw):
    g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                        wl.w_init, nu=wl.nu, rho=wl.rho, **kw)
    try:
        g.step(passes)
        L = len(wl.widths) - 1
        out = dict(dec=g.decisions(), obj=g.objective(), U=g.get_state(binding.ST_U))
        for l in range(1, L + 1):
            out[f"W{l}"] = g.get_state(binding.ST_W, l)
            out[f"Z{l}"] = g.get_state(binding.ST_Z, l)
            out[f"tau{l}"] = g.get_state(binding.ST_TAU, l)
        for l in range(1, L):
            out[f"theta{l}"] = g.get_state(binding.ST_THETA, l)
        return out
    finally:
        g.destroy()


@pytest.mark.parametrize("name,make_wl,kw", [
    ("cfg0", lambda: inputs.make_workload(0), {}),
    ("cfg3@0.012", lambda: inputs.make_workload(3, scale=0.012), {}),
    ("cfg3@0.05 cut rows", lambda: inputs.make_workload(3, scale=0.05), dict(long_row=16)),
    ("cfg2@0.3 serial", lambda: inputs.make_workload(2, scale=0.3), dict(schedule=1)),
], ids=lambda c: c if isinstance(c, str) else "")
def test_ten_passes_twice_bit_for_bit(name, make_wl, kw):
    wl = make_wl()
    a, b = run(wl, 10, **kw), run(wl, 10, **kw)
    for key in a:
        if key == "dec":
            for part in ("trial_w", "trial_z", "q_w", "q_z"):
                assert np.array_equal(a["dec"][part], b["dec"][part]), (name, part)
        else:
            assert np.array_equal(a[key], b[key]), (name, key)
