"""Host-side checks of the C-ABI library that need no GPU: it builds, loads, exports every
symbol the header declares, validates its inputs before touching CUDA and fails loudly
(no CPU fallback) when no device is present."""
import os
import re

import numpy as np
import pytest

from conftest import dense_to_csr, random_graph
from paper_2112_09335_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "gcn_admm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(gcn_admm_[a-z_0-9]+)\s*\(", text))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_default_params(lib):
    p = binding.default_params()
    assert abs(p.nu - 1e-3) < 1e-9 and abs(p.rho - 1e-3) < 1e-9
    assert p.bt_max_trials == 40 and p.fista_iters == 30 and p.dual_mode == 0
    assert p.bt_growth == 2.0 and p.bt_shrink == 0.5 and p.tau0 == 1.0 and p.theta0 == 1.0


def problem(seed=0, n=12):
    rng = np.random.default_rng(seed)
    row_ptr, col_idx, A = random_graph(rng, n, 0.3)
    return dict(n=n, row_ptr=row_ptr, col_idx=col_idx, X=rng.standard_normal((n, 4)).astype(np.float32),
                y=rng.integers(0, 3, n).astype(np.int32), train_mask=np.ones(n, dtype=np.uint8), widths=[4, 5, 3],
                n_comm=2, community=(np.arange(n) % 2).astype(np.int32),
                w_init=[rng.standard_normal((4, 5)).astype(np.float32), rng.standard_normal((5, 3)).astype(np.float32)])


def expect_error(code, **override):
    kw = problem()
    kw.update(override)
    with pytest.raises(binding.GcnAdmmError) as e:
        binding.GcnAdmm(**kw)
    assert e.value.code == code, str(e.value)


def test_input_validation_happens_on_the_host(lib):
    pr = problem()
    col = pr["col_idx"].copy()
    col[0] = pr["n"] + 5
    expect_error(-2, col_idx=col)                                   # column out of range
    rp, ci, A = pr["row_ptr"], pr["col_idx"], None
    first = int(np.flatnonzero(np.diff(rp) >= 2)[0])
    swapped = ci.copy()
    swapped[rp[first]], swapped[rp[first] + 1] = ci[rp[first] + 1], ci[rp[first]]
    expect_error(-2, col_idx=swapped)                               # unsorted row
    A = np.zeros((12, 12)); A[0, 1] = 1                             # asymmetric
    rp2, ci2 = dense_to_csr(A)
    expect_error(-2, row_ptr=rp2, col_idx=ci2)
    bad_rp = rp.copy(); bad_rp[3] = bad_rp[2] - 1
    expect_error(-2, row_ptr=bad_rp)                                # row_ptr not ascending
    expect_error(-3, community=np.full(12, 7, dtype=np.int32))      # id out of range
    expect_error(-3, community=np.zeros(12, dtype=np.int32))        # community 1 empty
    expect_error(-4, widths=[4, 0, 3])                              # zero width
    expect_error(-4, y=np.full(12, 9, dtype=np.int32))              # label outside 0..C_L-1
    expect_error(-1, nu=-1.0)
    expect_error(-1, bt_growth=1.0)
    expect_error(-1, bt_max_trials=0)


def test_no_cpu_fallback_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.GcnAdmmError) as e:
        binding.GcnAdmm(**problem())
    assert e.value.code == -6


def test_null_handle_is_rejected(lib):
    import ctypes as C
    assert lib.gcn_admm_step(None, 1) == -1
    out = (C.c_double * 6)()
    assert lib.gcn_admm_objective(None, out) == -1
    lib.gcn_admm_destroy(None)
