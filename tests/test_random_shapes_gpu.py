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


# ---- seeded random CHAINS conv -> pool -> conv: whatever the stack decides (staged hand-off, pool in the epilogue or as a
# kernel, first-layer kernel) must reproduce the fp64 oracle chain EXACTLY on operands from {-1, 0, 1}
def _chains(seed, count):
    r = wl.uniform01(seed, count * 10).reshape(count, 10)
    out = []
    for u in r:
        pick = lambda a, lst: lst[min(int(a * len(lst)), len(lst) - 1)]
        first_layer = u[0] < 0.4
        N = pick(u[1], [1, 2, 3])
        if first_layer:            # 3 channels, stride 4, no padding: legal for the first-layer kernel
            R = pick(u[2], [5, 7, 8, 9, 11]); S = R if u[3] < 0.6 else pick(u[3], [5, 7, 9, 11])
            P = pick(u[4], [7, 9, 12, 15, 21]); Q = pick(u[5], [7, 10, 13, 15, 22])
            c1 = wl.ConvShape(N, 3, 4 * (P - 1) + R, 4 * (Q - 1) + S, pick(u[6], [16, 40, 64, 96]), R, S, 4, 0, True)
        else:
            R = pick(u[2], [2, 3, 3, 5]); pad = pick(u[3], [0, 1, 1, 2]); pad = min(pad, R - 1)
            H = pick(u[4], [7, 9, 13, 16, 19]); W = pick(u[5], [7, 10, 13, 17, 20])
            c1 = wl.ConvShape(N, pick(u[6], [8, 24, 40, 64]), H, W, pick(u[7], [16, 40, 72, 96]), R, R, 1, pad, True)
        if c1.P < 3 or c1.Q < 3:
            continue
        pP, pQ = (c1.P - 3) // 2 + 1, (c1.Q - 3) // 2 + 1
        R2 = pick(u[8], [1, 3, 3, 5]); pad2 = R2 // 2
        c2 = wl.ConvShape(N, c1.K, pP, pQ, pick(u[9], [16, 48, 80]), R2, R2, 1, pad2, False)
        out.append((c1, c2, first_layer))
    return out


CHAINS = _chains(0xC4A1, 40)


@pytest.mark.parametrize("idx", range(len(CHAINS)))
@pytest.mark.parametrize("forced", [False, True])
def test_random_chain_exact(idx, forced):
    """forced: the first convolution on a tile that can run the pool in its epilogue (a halo tile, or the first-layer
    kernel), where the library accepts it for the shape; otherwise the rules choose."""
    import torch
    from oracle import conv_oracle as orc
    from paper_1606_00094_b200 import binding as B
    from paper_1606_00094_b200.stack import ConvStack
    c1, c2, first_layer = CHAINS[idx]
    ops = [wl.StackOp("conv", c1), wl.StackOp("pool"), wl.StackOp("conv", c2)]
    tern = lambda seed, shape: wl.integers(seed, shape, -1, 1)
    x = tern(9000 + idx, (c1.N, c1.C, c1.H, c1.W))
    # sparse second-layer filters keep every sum far below 2^24; the first layer's sums are at most C*R*S <= 2048
    w2 = (tern(9300 + idx, (c2.K, c2.C, c2.R, c2.S)) * (wl.uniform01(9400 + idx, c2.K * c2.C * c2.R * c2.S).reshape(c2.K, c2.C, c2.R, c2.S) < 0.2)).astype(np.float32)
    params = [(tern(9100 + idx, (c1.K, c1.C, c1.R, c1.S)), tern(9200 + idx, (c1.K,))), (w2, tern(9500 + idx, (c2.K,)))]
    assert c1.C * c1.R * c1.S + 1 <= 2048
    a = orc.conv_fwd(x, params[0][0], params[0][1], stride=c1.stride, pad=c1.pad, relu=True)
    pooled = orc.maxpool_fwd(a, 3, 2)
    ref = orc.conv_fwd(pooled, params[1][0], params[1][1], stride=1, pad=c2.pad, relu=False)
    per_op = None
    if forced:
        per_op = [{"variant": 2, "tile_id": 24 if first_layer else 10}, {}, {}]
    try:
        stack = ConvStack(ops, params, per_op=per_op)
    except B.BodaError as e:
        assert forced and e.status == B.BODA_ERR_UNSUPPORTED, f"{c1} {c2}: {e}"
        pytest.skip("the forced tile does not take this shape")
    try:
        descs = stack.describe()
        out = stack.forward(torch.from_numpy(x).cuda())
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0
        got_pool = stack.layer_output(1)
        np.testing.assert_array_equal(got_pool.cpu().numpy().astype(np.float64), pooled, err_msg=str(descs))
        np.testing.assert_array_equal(out.cpu().numpy().astype(np.float64), ref, err_msg=str(descs))
    finally:
        stack.close()
