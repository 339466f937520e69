"""Failure detection without a fault: a bounded wait inside the tensor-core kernels runs out and is reported.

A test hook makes the producer of ONE CTA announce 16 bytes more than its TMA loads deliver, so that CTA's
"stage full" barrier never completes.  The wait gives up after its cycle limit (shortened here), the kernel
records BODA_ERR_DEVICE_TIMEOUT in the status word, every role leaves its loop, tensor memory is released and the
kernel returns; the context stays usable, which the second half of the test checks with a normal run.
"""
import os

import numpy as np
import pytest

from paper_1606_00094_b200 import workloads as wl
from helpers import TF32_TOL, assert_parity, oracle_out

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("tile,split", [(2, 1), (6, 1), (3, 2), (10, 2), (17, 1)])   # im2col and halo kernels, with and without a cluster; gather kernel
def test_expired_wait_sets_status_and_context_survives(tile, split):
    import torch
    from paper_1606_00094_b200 import binding as B
    shape = (3, 64, 13, 13, 200, 3, 3, 1, 1, 1)
    N, C, H, W, K, R, S, st, pad, relu = shape
    x = wl.half_normal(1, (N, C, H, W))
    w = wl.normal(2, (K, C, R, S), 0, (2.0 / (C * R * S)) ** 0.5)
    b = wl.normal(3, (K,), 0, 0.01)
    dx, dw, db = (torch.from_numpy(t).cuda() for t in (x, w, b))
    assert B.boda_query_status() == 0
    os.environ["BODA_TEST_TX_MISMATCH"] = "1"
    os.environ["BODA_WAIT_LIMIT_CYCLES"] = "100000000"          # about 50 ms
    try:
        plan = B.ConvPlan(shape, variant=B.BODA_VARIANT_TCONV, tile_id=tile, split_k=split)
    finally:
        del os.environ["BODA_TEST_TX_MISMATCH"]
        del os.environ["BODA_WAIT_LIMIT_CYCLES"]
    plan(dx, dw, db)
    torch.cuda.synchronize()                                    # the kernel returns by itself
    assert B.boda_query_status() == B.BODA_ERR_DEVICE_TIMEOUT
    assert B.boda_query_status() == 0                           # reading the word clears it
    plan.close()
    # the same layer without the hook: correct result, clean status
    plan = B.ConvPlan(shape, variant=B.BODA_VARIANT_TCONV, tile_id=tile, split_k=split)
    got = plan(dx, dw, db).cpu().numpy()
    torch.cuda.synchronize()
    assert B.boda_query_status() == 0
    plan.close()
    assert_parity(got, oracle_out(shape, x, w, b), TF32_TOL)


@pytest.mark.parametrize("split", [1, 2])          # persistent form, and one tile per CTA with a cluster split over the channels
def test_expired_wait_in_the_nchw_1x1_kernel(split):
    import torch
    from paper_1606_00094_b200 import binding as B
    shape = (3, 64, 12, 12, 200, 1, 1, 1, 0, 1)
    N, C, H, W, K, R, S, st, pad, relu = shape
    x = wl.half_normal(4, (N, C, H, W))
    w = wl.normal(5, (K, C, R, S), 0, (2.0 / C) ** 0.5)
    b = wl.normal(6, (K,), 0, 0.01)
    dx, dw, db = (torch.from_numpy(t).cuda() for t in (x, w, b))
    assert B.boda_query_status() == 0
    os.environ["BODA_TEST_TX_MISMATCH"] = "1"
    os.environ["BODA_WAIT_LIMIT_CYCLES"] = "100000000"
    try:
        plan = B.ConvPlan(shape, variant=B.BODA_VARIANT_K1CONV, tile_id=20, split_k=split)
    finally:
        del os.environ["BODA_TEST_TX_MISMATCH"]
        del os.environ["BODA_WAIT_LIMIT_CYCLES"]
    plan(dx, dw, db)
    torch.cuda.synchronize()
    assert B.boda_query_status() == B.BODA_ERR_DEVICE_TIMEOUT
    assert B.boda_query_status() == 0
    plan.close()
    plan = B.ConvPlan(shape, variant=B.BODA_VARIANT_K1CONV, tile_id=20, split_k=split)
    got = plan(dx, dw, db).cpu().numpy()
    torch.cuda.synchronize()
    assert B.boda_query_status() == 0
    plan.close()
    assert_parity(got, oracle_out(shape, x, w, b), TF32_TOL)


def test_expired_wait_in_the_first_layer_kernel():
    import torch
    from paper_1606_00094_b200 import binding as B
    shape = (2, 3, 67, 67, 80, 11, 11, 4, 0, 1)
    N, C, H, W, K, R, S, st, pad, relu = shape
    x = wl.half_normal(7, (N, C, H, W))
    w = wl.normal(8, (K, C, R, S), 0, (2.0 / (C * R * S)) ** 0.5)
    b = wl.normal(9, (K,), 0, 0.01)
    dx, dw, db = (torch.from_numpy(t).cuda() for t in (x, w, b))
    assert B.boda_query_status() == 0
    os.environ["BODA_TEST_TX_MISMATCH"] = "1"
    os.environ["BODA_WAIT_LIMIT_CYCLES"] = "100000000"
    try:
        plan = B.ConvPlan(shape, variant=B.BODA_VARIANT_TCONV, tile_id=24)
    finally:
        del os.environ["BODA_TEST_TX_MISMATCH"]
        del os.environ["BODA_WAIT_LIMIT_CYCLES"]
    plan(dx, dw, db)
    torch.cuda.synchronize()
    assert B.boda_query_status() == B.BODA_ERR_DEVICE_TIMEOUT
    assert B.boda_query_status() == 0
    plan.close()
    plan = B.ConvPlan(shape, variant=B.BODA_VARIANT_TCONV, tile_id=24)
    got = plan(dx, dw, db).cpu().numpy()
    torch.cuda.synchronize()
    assert B.boda_query_status() == 0
    plan.close()
    assert_parity(got, oracle_out(shape, x, w, b), TF32_TOL)
