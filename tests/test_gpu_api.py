"""Behaviour of the C ABI on a GPU beyond the numerics: inputs given as device pointers, argument
checks that need a live handle, non-finite detection, two handles side by side, the launch counter."""
import numpy as np
import pytest

from paper_2112_09335_b200 import binding, inputs
from parity_utils import relerr

pytestmark = pytest.mark.gpu


def make(wl, **kw):
    return binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                           wl.w_init, nu=wl.nu, rho=wl.rho, **kw)


def test_create_from_device_pointers_equals_create_from_host():
    import torch
    wl = inputs.make_workload(1)
    t = dict(row_ptr=torch.from_numpy(wl.row_ptr).cuda(), col_idx=torch.from_numpy(wl.col_idx).cuda(),
             X=torch.from_numpy(wl.X).cuda(), y=torch.from_numpy(wl.y).cuda(),
             mask=torch.from_numpy(wl.train_mask).cuda(), comm=torch.from_numpy(wl.community).cuda())
    a = make(wl)
    b = binding.GcnAdmm(wl.n, t["row_ptr"].data_ptr(), t["col_idx"].data_ptr(), t["X"].data_ptr(), t["y"].data_ptr(),
                        t["mask"].data_ptr(), wl.widths, wl.n_comm, t["comm"].data_ptr(), wl.w_init, nu=wl.nu, rho=wl.rho)
    try:
        a.step(3)
        b.step(3)
        for l in range(1, len(wl.widths)):
            assert np.array_equal(a.get_state(binding.ST_W, l), b.get_state(binding.ST_W, l))
            assert relerr(a.get_state(binding.ST_Z, l), b.get_state(binding.ST_Z, l)) < 1e-6
    finally:
        a.destroy()
        b.destroy()


def test_argument_checks_on_a_live_handle():
    wl = inputs.make_workload(0)
    g = make(wl)
    try:
        L = len(wl.widths) - 1
        for call in (lambda: g.step(-1), lambda: g.step_block(binding.PHASE_W, 0), lambda: g.step_block(binding.PHASE_Z, L + 1),
                     lambda: g.step_block(7, 1), lambda: g.weights(L + 1), lambda: g.get_state(binding.ST_THETA, L),
                     lambda: g.set_state(binding.ST_TAU, 1, np.array([-1.0])), lambda: g.index("nbr", wl.n_comm)):
            with pytest.raises(binding.GcnAdmmError) as e:
                call()
            assert e.value.code == -1, str(e.value)
        g.step(1)                      # the handle stays usable after rejected calls
        assert np.isfinite(g.objective()).all()
    finally:
        g.destroy()


def test_non_finite_input_is_reported():
    wl = inputs.make_workload(0)
    X = wl.X.copy()
    X[3, 5] = np.nan
    g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                        wl.w_init, nu=wl.nu, rho=wl.rho)
    try:
        g.step(3)
        with pytest.raises(binding.GcnAdmmError) as e:
            g.decisions()
        assert e.value.code == -7, str(e.value)
    finally:
        g.destroy()


def test_two_handles_do_not_interfere_and_launches_are_counted():
    wl0, wl1 = inputs.make_workload(0), inputs.make_workload(2, scale=0.1)
    a, b, ref = make(wl0), make(wl1), make(wl0)
    try:
        before = a.launches()
        a.step(2)
        b.step(2)
        a.step(2)
        ref.step(4)
        assert a.launches() > before
        for l in range(1, len(wl0.widths)):
            assert relerr(a.get_state(binding.ST_Z, l), ref.get_state(binding.ST_Z, l)) < 1e-6
    finally:
        a.destroy()
        b.destroy()
        ref.destroy()
