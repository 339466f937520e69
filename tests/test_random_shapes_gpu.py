"""Seeded random layer shapes through every variant that accepts them, against the fp64 oracle.

The hand-picked cases of the other files aim at known tile and padding boundaries; this sweep looks for the
ones nobody thought of: ragged channel counts, windows larger than the image plus padding allows elsewhere,
strides that do not divide, one-pixel outputs, R != S.  Outputs sit between NaN guard bands."""
import numpy as np
import pytest

from paper_1606_00094_b200 import workloads as wl
from helpers import FP32_TOL, TF32_TOL, assert_parity, oracle_out, run_planned

pytestmark = pytest.mark.gpu

DIRECT, K1, TC = 0, 1, 2


def _shapes(seed, count):
    r = wl.uniform01(seed, count * 12).reshape(count, 12)
    out = []
    for u in r:
        pick = lambda a, lst: lst[min(int(a * len(lst)), len(lst) - 1)]
        N = pick(u[0], [1, 1, 2, 3, 5])
        C = pick(u[1], [1, 3, 4, 8, 16, 20, 32, 33, 48, 64, 96, 100])
        K = pick(u[2], [1, 8, 16, 17, 24, 32, 64, 96, 130, 200])
        R = pick(u[3], [1, 1, 2, 3, 3, 4, 5, 7])
        S = R if u[4] < 0.7 else pick(u[5], [1, 2, 3, 5])
        stride = pick(u[6], [1, 1, 1, 2, 2, 3, 4])
        pad = pick(u[7], [0, 0, 1, 1, 2, 3])
        H = max(R - 2 * pad, 1) + pick(u[8], [0, 1, 2, 5, 9, 14, 23])
        W = max(S - 2 * pad, 1) + pick(u[9], [0, 1, 3, 6, 11, 17, 30])
        relu = 1 if u[10] < 0.5 else 0
        out.append((N, C, H, W, K, R, S, stride, pad, relu))
    return out


def _tensors(shape, seed):
    N, C, H, W, K, R, S, st, pad, relu = shape
    return (wl.normal(seed, (N, C, H, W)), wl.normal(seed + 1, (K, C, R, S), 0, (2.0 / (C * R * S)) ** 0.5),
            wl.normal(seed + 2, (K,), 0, 0.1))


SHAPES = _shapes(0x51AE5, 60)


@pytest.mark.parametrize("idx", range(len(SHAPES)))
def test_random_shape_all_variants(idx):
    from paper_1606_00094_b200 import binding as B
    shape = SHAPES[idx]
    x, w, b = _tensors(shape, 7000 + 10 * idx)
    ref = oracle_out(shape, x, w, b)
    ran = 0
    # (variant, math, tolerance); forced variants that the library refuses for the shape are skipped, not failed
    for variant, math, tol in ((-1, 0, TF32_TOL), (DIRECT, 1, FP32_TOL), (K1, 2, TF32_TOL), (TC, 2, TF32_TOL), (-1, 3, FP32_TOL)):
        try:
            got, desc = run_planned(shape, x, w, b, variant=variant, math=math)
        except B.BodaError as e:
            assert e.status in (B.BODA_ERR_UNSUPPORTED,), f"{shape} variant {variant} math {math}: {e}"
            continue
        assert got.shape == ref.shape
        assert_parity(got, ref, tol, f"{shape} {desc}")
        ran += 1
    assert ran >= 2, f"{shape}: only {ran} variants ran"


@pytest.mark.parametrize("idx", range(0, len(SHAPES), 2))
def test_random_shape_forced_tiles_splits_and_views(idx):
    """The same shapes through tiles the cost model would not pick: a halo tile of each accumulator count, a
    split reduction, and the space-to-depth view; whatever the library accepts must meet the bar."""
    from paper_1606_00094_b200 import binding as B
    shape = SHAPES[idx]
    if shape[5] * shape[6] < 2:
        pytest.skip("1x1 layers have one tensor-core kernel")
    x, w, b = _tensors(shape, 7000 + 10 * idx)
    ref = oracle_out(shape, x, w, b)
    ran = 0
    for kw in (dict(tile_id=6), dict(tile_id=10), dict(tile_id=14), dict(tile_id=1, split_k=3), dict(tile_id=3, split_k=8),
               dict(s2d=1), dict(tile_id=9, s2d=1)):
        try:
            got, desc = run_planned(shape, x, w, b, variant=TC, math=2, **kw)
        except B.BodaError as e:
            assert e.status == B.BODA_ERR_UNSUPPORTED, f"{shape} {kw}: {e}"
            continue
        assert_parity(got, ref, TF32_TOL, f"{shape} {desc}")
        ran += 1
    assert ran >= 1


# the degenerate corners, by hand: one element of everything, one-pixel outputs, windows as large as the image, strides
# larger than the window, rows and columns of one pixel, padding that makes the border outputs pure bias
DEGENERATE = [
    (1, 1, 1, 1, 1, 1, 1, 1, 0, 0),
    (1, 1, 3, 3, 1, 3, 3, 1, 0, 1),
    (2, 5, 4, 4, 3, 2, 2, 3, 0, 0),
    (1, 2, 1, 9, 4, 1, 3, 1, 1, 1),
    (1, 2, 9, 1, 4, 3, 1, 2, 1, 0),
    (3, 7, 5, 5, 2, 5, 5, 1, 2, 1),
    (1, 4, 2, 2, 5, 1, 1, 1, 3, 0),
    (4, 1, 8, 8, 1, 1, 1, 8, 0, 1),
]


@pytest.mark.parametrize("shape", DEGENERATE)
def test_degenerate_shapes_exact_on_integers(shape):
    from paper_1606_00094_b200 import binding as B
    N, C, H, W, K, R, S, st, pad, relu = shape
    x, w, b = wl.integers(8100, (N, C, H, W)), wl.integers(8101, (K, C, R, S)), wl.integers(8102, (K,))
    ref = oracle_out(shape, x, w, b)
    ran = 0
    for variant, math in ((-1, 0), (DIRECT, 1), (K1, 2), (TC, 2), (-1, 3)):
        try:
            got, desc = run_planned(shape, x, w, b, variant=variant, math=math)
        except B.BodaError as e:
            assert e.status == B.BODA_ERR_UNSUPPORTED, f"{shape} variant {variant} math {math}: {e}"
            continue
        np.testing.assert_array_equal(got.astype(np.float64), ref, err_msg=f"{shape} {desc}")
        ran += 1
    assert ran >= 2
