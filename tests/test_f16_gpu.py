"""GPU parity of the reduced-precision storage mode (fp16 operands, fp32 accumulation on the tensor cores).

Two bars, both against the fp64 oracle: (i) with the oracle fed the SAME fp16-rounded operands the only error left is
the fp32 accumulation, so the FP32 bar (1e-5) applies - products of two fp16 values are exact in fp32; (ii) with the
oracle fed the original fp32 operands the operand rounding (10 mantissa bits, like TF32) shows and the TF32 bar (5e-3)
applies.  Integer operands are exact in fp16, so those results must match bit for bit.
"""
import numpy as np
import pytest

from paper_1606_00094_b200 import workloads as wl
from helpers import FP32_TOL, TF32_TOL, assert_parity, oracle_out, run_planned

pytestmark = pytest.mark.gpu

F16 = 4         # BODA_MATH_F16
K1, TC = 1, 2


def _real_tensors(shape, seed):
    N, C, H, W, K, R, S, st, pad, relu = shape
    return (wl.half_normal(seed, (N, C, H, W)), wl.normal(seed + 1, (K, C, R, S), 0, (2.0 / (C * R * S)) ** 0.5),
            wl.normal(seed + 2, (K,), 0, 0.01))


def _as_fp16(a):
    """The value the staging kernels store: round to nearest even fp16, widened back."""
    return a.astype(np.float16).astype(np.float32)


CASES = [
    ((5, 480, 14, 14, 192, 1, 1, 1, 0, 1), K1),         # configuration 3
    ((4, 256, 13, 13, 384, 3, 3, 1, 1, 1), TC),         # configuration 4 at batch 4
    ((2, 96, 27, 27, 256, 5, 5, 1, 2, 1), TC),          # conv2-like (96 channels: padded to 128 = two chunks of 64)
    ((3, 50, 20, 20, 70, 3, 3, 2, 1, 0), TC),           # stride 2, ragged channels and tiles, no ReLU
    ((1, 3, 227, 227, 96, 11, 11, 4, 0, 1), TC),        # configuration 2: three input channels, stride 4
    ((2, 40, 9, 11, 24, 3, 5, 1, 2, 0), TC),            # R != S, single tile
]


@pytest.mark.parametrize("shape,variant", CASES)
def test_both_bars(shape, variant):
    x, w, b = _real_tensors(shape, 2300)
    ref_rounded = oracle_out(shape, _as_fp16(x), _as_fp16(w), b)       # the bias stays fp32 (added in the epilogue)
    ref = oracle_out(shape, x, w, b)
    for bind in (False, True):
        got, desc = run_planned(shape, x, w, b, variant=variant, math=F16, bind=bind)
        assert "math=f16" in desc and " f16 " in desc, desc
        assert_parity(got, ref_rounded, FP32_TOL, desc + " (fp16-rounded operands)")
        assert_parity(got, ref, TF32_TOL, desc)


@pytest.mark.parametrize("tile", range(5))
@pytest.mark.parametrize("split", [1, 2, 4])
def test_every_im2col_tile_and_split_exact(tile, split):
    shape = (3, 72, 13, 13, 272, 3, 3, 1, 1, 1)          # 72 channels: the second chunk of 64 is mostly padding
    x, w, b = wl.integers(2400, (3, 72, 13, 13)), wl.integers(2401, (272, 72, 3, 3)), wl.integers(2402, (272,))
    got, desc = run_planned(shape, x, w, b, variant=TC, math=F16, tile_id=tile, split_k=split)
    assert f"id {tile}" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_auto_variant_and_k1conv_exact():
    shape = (2, 100, 14, 14, 48, 1, 1, 1, 0, 0)
    x, w, b = wl.integers(2500, (2, 100, 14, 14)), wl.integers(2501, (48, 100, 1, 1)), wl.integers(2502, (48,))
    got, desc = run_planned(shape, x, w, b, math=F16)
    assert "variant=k1conv" in desc and "math=f16" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_never_chosen_automatically_and_other_kernels_refused():
    import torch  # noqa: F401  (the binding needs a device)
    from paper_1606_00094_b200 import binding as B
    plan = B.ConvPlan((4, 256, 13, 13, 384, 3, 3, 1, 1, 1))
    assert "math=tf32" in plan.describe()
    plan.close()
    with pytest.raises(Exception):
        B.ConvPlan((2, 64, 13, 13, 64, 3, 3, 1, 1, 1), math=F16, variant=TC, tile_id=5)      # a halo tile
    with pytest.raises(Exception):
        B.ConvPlan((1, 3, 227, 227, 96, 11, 11, 4, 0, 1), math=F16, variant=TC, s2d=1)
