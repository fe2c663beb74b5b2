"""The dense product C = A B of the library (tensor-core path: error-compensated TF32 with fp32
accumulation; fp32 FMA path) against numpy in fp64, through the C ABI, on shapes with ragged tails."""
import numpy as np
import pytest

from paper_2112_09335_b200 import binding, inputs

pytestmark = pytest.mark.gpu

SHAPES = [(1000, 16, 128), (5000, 256, 256), (4097, 256, 100), (3000, 47, 256), (2049, 16, 1433), (700, 5, 37),
          (130, 256, 8), (40000, 128, 500), (33000, 256, 256), (20001, 47, 256), (16384, 256, 100), (777, 3, 128), (12345, 40, 256), (9000, 1000, 767), (6000, 10, 1000), (3000, 300, 64),
          (17001, 200, 47), (16500, 130, 128), (16390, 129, 33)]    # (m, n, k); the last three: two groups of 128 columns, the second one ragged


@pytest.fixture(scope="module")
def handle():
    wl = inputs.make_workload(3, scale=0.02)     # wide layers: room for many row splits of the transposed product
    g = binding.GcnAdmm(wl.n, wl.row_ptr, wl.col_idx, wl.X, wl.y, wl.train_mask, wl.widths, wl.n_comm, wl.community,
                        wl.w_init)
    yield g
    g.destroy()


@pytest.mark.parametrize("tensor_cores", [1, 2, 0])     # 2: weight operand pre-split at every size (1 does so from 16384 rows)
@pytest.mark.parametrize("m,n,k", SHAPES)
def test_dense_product_against_fp64(handle, m, n, k, tensor_cores):
    import torch
    rng = np.random.default_rng(m + n + k)
    a = rng.standard_normal((m, k)).astype(np.float32)
    b = (rng.standard_normal((k, n)) * rng.choice([1e-3, 1.0, 30.0], size=(1, n))).astype(np.float32)
    ta, tb = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    tc = torch.full((m, n), float("nan"), device="cuda")
    handle.dense_product(ta.data_ptr(), tb.data_ptr(), tc.data_ptr(), m, n, k, tensor_cores)
    got = tc.cpu().numpy().astype(np.float64)
    want = a.astype(np.float64) @ b.astype(np.float64)
    scale = np.abs(a).astype(np.float64) @ np.abs(b).astype(np.float64) + 1e-300
    worst = float(np.max(np.abs(got - want) / scale))
    rel = float(np.linalg.norm(got - want) / np.linalg.norm(want))
    print(f"\n  m={m} n={n} k={k} tc={tensor_cores}: rel {rel:.2e}, worst elementwise/sum|a||b| {worst:.2e}")
    assert np.isfinite(got).all()
    assert worst < 2e-6
    assert rel < 3e-6 * max(1.0, k / 512)      # the tensor core's accumulator error grows with K


TN_SHAPES = [(50000, 128, 16), (30011, 256, 256), (20000, 100, 256), (40001, 256, 47), (8192, 128, 7), (100000, 16, 7),
             (4096, 300, 40), (5000, 37, 129), (13752, 767, 1000), (13752, 1000, 10)]    # (rows, ka, nb)


@pytest.mark.parametrize("tensor_cores", [1, 0])
@pytest.mark.parametrize("rows,ka,nb", TN_SHAPES)
def test_transposed_product_against_fp64(handle, rows, ka, nb, tensor_cores):
    import torch
    rng = np.random.default_rng(rows + ka + nb)
    a = rng.standard_normal((rows, ka)).astype(np.float32)
    b = (rng.standard_normal((rows, nb)) * rng.choice([1e-3, 1.0, 30.0], size=(1, nb))).astype(np.float32)
    ta, tb = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    tc = torch.full((ka, nb), float("nan"), device="cuda")
    handle.dense_product_tn(ta.data_ptr(), tb.data_ptr(), tc.data_ptr(), rows, ka, nb, tensor_cores)
    got = tc.cpu().numpy().astype(np.float64)
    want = a.astype(np.float64).T @ b.astype(np.float64)
    scale = np.abs(a).astype(np.float64).T @ np.abs(b).astype(np.float64) + 1e-300
    worst = float(np.max(np.abs(got - want) / scale))
    rel = float(np.linalg.norm(got - want) / np.linalg.norm(want))
    print(f"\n  rows={rows} ka={ka} nb={nb} tc={tensor_cores}: rel {rel:.2e}, worst elementwise/sum|a||b| {worst:.2e}")
    assert np.isfinite(got).all()
    assert worst < 2e-6
    assert rel < 2e-4      # the sum over many rows cancels: relative to ||C|| the bound is loose, `worst` is the sharp one
