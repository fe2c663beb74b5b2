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


def splitmix64(x):
    """Output function of the splitmix64 generator at state x + 0x9E3779B97F4A7C15 (Steele, Lea, Flood 2014)."""
    m = (1 << 64) - 1
    z = (x + 0x9E3779B97F4A7C15) & m
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    return z ^ (z >> 31)


def test_seeded_initial_weights_when_none_are_given():
    """w_init = NULL: Glorot-uniform from the counter-based generator the header defines, re-derived here."""
    wl = inputs.make_workload(0)
    def weights(seed):
        g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                            None, nu=wl.nu, rho=wl.rho, seed=seed)
        try:
            g.step(2)                                                   # the handle works like any other
            assert np.isfinite(g.objective()).all()
            g2 = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm,
                                 wl.community, None, nu=wl.nu, rho=wl.rho, seed=seed)
            try:
                return [g2.weights(l) for l in range(1, len(wl.widths))]
            finally:
                g2.destroy()
        finally:
            g.destroy()
    a, b = weights(12345), weights(12346)
    for l, w in enumerate(a, start=1):
        r, c = wl.widths[l - 1], wl.widths[l]
        bound = np.sqrt(6.0 / (r + c))
        want = np.array([[bound * (2.0 * ((splitmix64(12345 + (l << 32) + i * c + j) >> 40) / 16777216.0) - 1.0)
                          for j in range(c)] for i in range(r)]).astype(np.float32)
        assert np.array_equal(w, want)
        assert np.abs(w).max() <= bound and abs(w.mean()) < 0.2 * bound
        assert not np.array_equal(w, b[l - 1])


def test_a_raised_pipeline_flag_surfaces_once_and_the_handle_stays_usable():
    """The bounded waits of the tensor-core products report through a device flag.  Host half of that path:
    with the flag written from here, the next synchronising call fails with GCN_ADMM_ERR_CUDA, the flag is
    cleared, and the handle keeps working."""
    wl = inputs.make_workload(0)
    g = make(wl)
    try:
        g.step(1)
        before = g.objective()
        g.set_state(binding.ST_PIPELINE_FLAG, 0, np.array([1], dtype=np.int32))
        with pytest.raises(binding.GcnAdmmError) as e:
            g.objective()
        assert e.value.code == -6 and "tensor-core" in str(e.value)
        assert int(g.get_state(binding.ST_PIPELINE_FLAG)[0]) == 0
        assert np.array_equal(g.objective(), before)
        g.step(1)
        assert np.isfinite(g.objective()).all()
    finally:
        g.destroy()


def test_shard_plan_through_the_library():
    """The multi-GPU plan (host logic, covered in depth on the CPU) as the library hands it out."""
    from oracle import gcn_admm_oracle as orc
    wl = inputs.make_workload(0)
    g = make(wl)
    try:
        R = 2
        ranges = g.shard_plan(R, 0)
        comm_begin, row_begin = ranges[:R + 1], ranges[R + 1:]
        ix = orc.community_index(wl.n, wl.row_ptr, wl.col_idx, wl.community, wl.n_comm)
        assert np.array_equal(row_begin, ix["comm_ptr"][comm_begin]) and comm_begin[0] == 0 and comm_begin[-1] == wl.n_comm
        for r in range(R):
            h1 = np.unique(np.concatenate([ix["halo1"][m] for m in range(comm_begin[r], comm_begin[r + 1])]))
            h1 = h1[(h1 < row_begin[r]) | (h1 >= row_begin[r + 1])]
            got = np.concatenate([g.shard_plan(R, 1, r, s) for s in range(R)])
            assert np.array_equal(np.sort(got), h1)
            assert len(g.shard_plan(R, 1, r, r)) == 0
        with pytest.raises(binding.GcnAdmmError):
            g.shard_plan(wl.n_comm + 1, 0)
    finally:
        g.destroy()
