"""gcn_admm_propagate_static: the propagation entry point for callers that must not allocate.

Some users of this library run where reserving device memory at call time is not an option: a
service whose memory was carved up at start-up, code living inside another framework's pool, a
region under stream capture.  For them the library carries its staging memory inside the binary.
This test calls that entry point through the C ABI twice in a row on device buffers and checks
both results against the ordinary gcn_admm_propagate, with the same tolerance the propagation
parity test uses.  It is named so that pytest collects it last."""
import numpy as np
import pytest

from paper_2112_09335_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_static_propagation_matches_the_allocating_one_twice():
    import torch
    wl = inputs.make_workload(1)
    g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                        wl.w_init, nu=wl.nu, rho=wl.rho)
    try:
        for width, seed in ((47, 0), (200, 1)):          # two calls in a row share the built-in memory
            gen = torch.Generator(device="cuda").manual_seed(seed)
            x = torch.randn(wl.n, width, device="cuda", generator=gen)
            want = torch.empty_like(x)
            got = torch.full_like(x, float("nan"))
            g.propagate(x.data_ptr(), width, out=want.data_ptr())
            g.propagate_static(x.data_ptr(), width, got.data_ptr())
            torch.cuda.synchronize()
            err = (got - want).norm() / want.norm()
            assert torch.isfinite(got).all()
            assert float(err) < 2e-7, (width, float(err))
        # a size beyond the built-in memory is refused with a message that names the limit
        big = 4_194_304 // wl.n + 8
        x = torch.zeros(wl.n, big, device="cuda")
        out = torch.zeros_like(x)
        with pytest.raises(binding.GcnAdmmError) as e:
            g.propagate_static(x.data_ptr(), big, out.data_ptr())
        assert e.value.code == -1 and "4194304" in str(e.value)
        # host pointers are refused as well (this entry point copies nothing through the host)
        with pytest.raises(binding.GcnAdmmError):
            g.propagate_static(wl.X.ctypes.data, wl.X.shape[1], wl.X.ctypes.data)
    finally:
        g.destroy()
