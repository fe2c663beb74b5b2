"""gcn_admm_step on a non-default stream replays a recorded CUDA graph of one pass; the result must be
the one plain launches give (same kernels, same order), and the decision log must still be per pass."""
import numpy as np
import pytest

from paper_2112_09335_b200 import binding, inputs
from parity_utils import relerr

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index,scale", [(0, 1.0), (3, 0.02)])
def test_graph_replay_matches_plain_launches(index, scale):
    import torch
    wl = inputs.make_workload(index, scale=scale)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        def make(use_graph):
            return binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm,
                                   wl.community, wl.w_init, nu=wl.nu, rho=wl.rho, stream=side.cuda_stream,
                                   use_graph=use_graph)
        a, b = make(1), make(0)
        try:
            a.step(4)
            a.step(6)            # second call replays the graph recorded by the first
            b.step(4)
            b.step(6)
            side.synchronize()
            da, db = a.decisions(), b.decisions()
            assert da["trial_w"].shape[0] == 6 and db["trial_w"].shape[0] == 6
            assert np.array_equal(da["trial_w"], db["trial_w"]) and np.array_equal(da["trial_z"], db["trial_z"])
            for l in range(1, len(wl.widths)):
                assert relerr(a.get_state(binding.ST_W, l), b.get_state(binding.ST_W, l)) < 1e-6
                assert relerr(a.get_state(binding.ST_Z, l), b.get_state(binding.ST_Z, l)) < 1e-6
            # the recorded pass forms every product; plain launches skip the H_1 = P_1 W_1 product that the W_1
            # step has already left behind (one launch per pass, here in all ten passes)
            assert a.launches() - b.launches() == 10
        finally:
            a.destroy()
            b.destroy()


def test_kept_first_layer_product_over_many_passes():
    """Plain launches keep H_1 = P_1 W_1 from the W_1 step and form it afresh only every 16th pass; a
    recorded graph forms it in every pass.  Over 36 passes (two refresh points) both must give the same
    iterates up to rounding."""
    import torch
    wl = inputs.make_workload(0)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        def make(use_graph):
            return binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm,
                                   wl.community, wl.w_init, nu=wl.nu, rho=wl.rho, stream=side.cuda_stream,
                                   use_graph=use_graph)
        a, b = make(1), make(0)
        try:
            a.step(36)
            b.step(36)
            side.synchronize()
            da, db = a.decisions(), b.decisions()
            assert np.array_equal(da["trial_w"], db["trial_w"]) and np.array_equal(da["trial_z"], db["trial_z"])
            for l in range(1, len(wl.widths)):
                assert relerr(a.get_state(binding.ST_W, l), b.get_state(binding.ST_W, l)) < 1e-5
                assert relerr(a.get_state(binding.ST_Z, l), b.get_state(binding.ST_Z, l)) < 1e-5
            assert a.launches() - b.launches() == 36 - 2      # passes 16 and 32 formed the product again
        finally:
            a.destroy()
            b.destroy()
