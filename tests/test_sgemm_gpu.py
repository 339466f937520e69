"""boda_sgemm (Section 4, Table 1: the paper's SGEMM warm-up) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import conv_oracle as orc
from paper_1606_00094_b200 import workloads as wl
from helpers import GUARD, TF32_TOL, assert_parity

pytestmark = pytest.mark.gpu


def _run(A, Bm):
    import torch
    from paper_1606_00094_b200 import binding as B
    M, K = A.shape
    N = Bm.shape[1]
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
    buf = torch.full((M * N + 2 * GUARD,), float("nan"), dtype=torch.float32, device="cuda")
    C = buf[GUARD:GUARD + M * N].view(M, N)
    B.boda_sgemm(dA, dB, C, M, N, K)
    torch.cuda.synchronize()
    assert B.boda_query_status() == 0
    host = buf.cpu().numpy()
    assert np.isnan(host[:GUARD]).all() and np.isnan(host[GUARD + M * N:]).all(), "guard band overwritten"
    out = host[GUARD:GUARD + M * N].reshape(M, N).copy()
    assert not np.isnan(out).any(), "output not fully written"
    return out


# Table 1 of the paper lists square problems 128 ... 2048 (the largest two are checked on sampled rows below)
@pytest.mark.parametrize("n", [128, 256, 384, 512, 768, 1024])
def test_table1_square_sizes(n):
    A = wl.normal(0x5601 + n, (n, n))
    Bm = wl.normal(0x5602 + n, (n, n))
    assert_parity(_run(A, Bm), orc.sgemm(A, Bm), TF32_TOL, f"sgemm {n}^3")


@pytest.mark.parametrize("n", [1536, 2048])
def test_table1_large_sizes_on_sampled_rows(n):
    A = wl.normal(0x5603 + n, (n, n))
    Bm = wl.normal(0x5604 + n, (n, n))
    got = _run(A, Bm)
    rows = wl.integers(0x5605 + n, (24,), 0, n - 1).astype(np.int64)
    rows = np.unique(np.concatenate([rows, np.array([0, 127, 128, n - 1])]))
    ref = orc.sgemm(A[rows], Bm)
    assert_parity(got[rows], ref, TF32_TOL, f"sgemm {n}^3 rows")


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (100, 77, 50), (130, 257, 33), (5, 300, 1000), (300, 5, 64), (129, 129, 129)])
def test_ragged_sizes(M, N, K):
    A = wl.normal(0x5611 + M, (M, K))
    Bm = wl.normal(0x5612 + N, (K, N))
    assert_parity(_run(A, Bm), orc.sgemm(A, Bm), TF32_TOL, f"sgemm {M}x{N}x{K}")


def test_integer_operands_are_exact():
    # small integers are exact in TF32 and every partial sum is exact in fp32: the result must match bit for bit
    M, N, K = 192, 160, 224
    A = wl.integers(0x5621, (M, K))
    Bm = wl.integers(0x5622, (K, N))
    np.testing.assert_array_equal(_run(A, Bm).astype(np.float64), orc.sgemm(A, Bm))


def test_rejects_bad_arguments():
    import torch
    from paper_1606_00094_b200 import binding as B
    t = torch.zeros(4, device="cuda")
    with pytest.raises(Exception):
        B.boda_sgemm(t, t, t, 0, 2, 2)
