"""GPU parity of the error-compensated TF32 mode (three tensor-core products per FP32 product) against the fp64
oracle: it must meet the FP32 bar, not the TF32 one."""
import numpy as np
import pytest

from paper_1606_00094_b200 import workloads as wl
from helpers import FP32_TOL, assert_parity, oracle_out, run_planned

pytestmark = pytest.mark.gpu

X3 = 3          # BODA_MATH_TF32X3
K1, TC = 1, 2


def _real_tensors(shape, seed):
    N, C, H, W, K, R, S, st, pad, relu = shape
    return (wl.half_normal(seed, (N, C, H, W)), wl.normal(seed + 1, (K, C, R, S), 0, (2.0 / (C * R * S)) ** 0.5),
            wl.normal(seed + 2, (K,), 0, 0.01))


CASES = [
    ((5, 480, 14, 14, 192, 1, 1, 1, 0, 1), K1),         # configuration 3
    ((4, 256, 13, 13, 384, 3, 3, 1, 1, 1), TC),         # configuration 4 at batch 4
    ((2, 96, 27, 27, 256, 5, 5, 1, 2, 1), TC),          # conv2-like
    ((3, 50, 20, 20, 70, 3, 3, 2, 1, 0), TC),           # stride 2, ragged channels and tiles, no ReLU
    ((1, 3, 227, 227, 96, 11, 11, 4, 0, 1), TC),        # configuration 2: three input channels, stride 4
    ((2, 40, 9, 11, 24, 3, 5, 1, 2, 0), TC),            # R != S, single tile
]


@pytest.mark.parametrize("shape,variant", CASES)
def test_meets_the_fp32_bar(shape, variant):
    x, w, b = _real_tensors(shape, 1300)
    ref = oracle_out(shape, x, w, b)
    for bind in (False, True):
        got, desc = run_planned(shape, x, w, b, variant=variant, math=X3, bind=bind)
        assert "math=tf32x3" in desc and " x3 " in desc, desc
        assert_parity(got, ref, FP32_TOL, desc)


@pytest.mark.parametrize("tile", range(5))
@pytest.mark.parametrize("split", [1, 2, 4])
def test_every_im2col_tile_and_split(tile, split):
    shape = (3, 64, 13, 13, 272, 3, 3, 1, 1, 1)
    x, w, b = _real_tensors(shape, 1400)
    got, desc = run_planned(shape, x, w, b, variant=TC, math=X3, tile_id=tile, split_k=split)
    assert f"id {tile}" in desc
    assert_parity(got, oracle_out(shape, x, w, b), FP32_TOL, desc)


def test_integers_exact_and_auto_variant():
    # integers are exact in TF32: their low parts are zero and the result must match bit for bit
    shape = (2, 64, 14, 14, 48, 3, 3, 1, 1, 1)
    x, w, b = wl.integers(1500, (2, 64, 14, 14)), wl.integers(1501, (48, 64, 3, 3)), wl.integers(1502, (48,))
    got, desc = run_planned(shape, x, w, b, math=X3)
    assert "variant=tconv" in desc and "tf32x3" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_much_closer_than_plain_tf32():
    shape = (4, 256, 13, 13, 384, 3, 3, 1, 1, 1)
    x, w, b = _real_tensors(shape, 1600)
    ref = oracle_out(shape, x, w, b)
    from oracle import conv_oracle as orc
    e1 = orc.rel_l2(run_planned(shape, x, w, b, variant=TC, math=2)[0], ref)
    e3 = orc.rel_l2(run_planned(shape, x, w, b, variant=TC, math=X3)[0], ref)
    assert e3 < e1 / 50, (e1, e3)


def test_halo_and_space_to_depth_are_refused():
    import torch  # noqa: F401  (the binding needs a device)
    from paper_1606_00094_b200 import binding as B
    with pytest.raises(Exception):
        B.ConvPlan((2, 64, 13, 13, 64, 3, 3, 1, 1, 1), math=X3, variant=TC, tile_id=5)      # a halo tile
    with pytest.raises(Exception):
        B.ConvPlan((1, 3, 227, 227, 96, 11, 11, 4, 0, 1), math=X3, variant=TC, s2d=1)
