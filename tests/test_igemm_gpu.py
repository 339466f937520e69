"""GPU parity of the tensor-core variants (K1CONV, TCONV: tcgen05 TF32 implicit GEMM) against the fp64 oracle."""
import numpy as np
import pytest

from paper_1606_00094_b200 import workloads as wl
from helpers import TF32_TOL, assert_parity, oracle_out, run_planned

pytestmark = pytest.mark.gpu

K1, TC = 1, 2


def _int_tensors(shape, seed):
    N, C, H, W, K, R, S, st, pad, relu = shape
    return wl.integers(seed, (N, C, H, W)), wl.integers(seed + 1, (K, C, R, S)), wl.integers(seed + 2, (K,))


def _real_tensors(shape, seed):
    N, C, H, W, K, R, S, st, pad, relu = shape
    return (wl.half_normal(seed, (N, C, H, W)), wl.normal(seed + 1, (K, C, R, S), 0, (2.0 / (C * R * S)) ** 0.5),
            wl.normal(seed + 2, (K,), 0, 0.01))


# integer-valued inputs in [-8, 8] are exact in TF32 and every partial sum is exact in fp32, so the
# tensor-core path must reproduce the oracle bit for bit: an indexing test that no tolerance can blur.
EXACT_CASES = [
    # shape, variant
    ((1, 32, 8, 8, 16, 1, 1, 1, 0, 0), K1),            # single tile, single chunk
    ((2, 64, 14, 14, 48, 1, 1, 1, 0, 1), K1),          # several pixel tiles, ragged last tile (392 = 3*128 + 8)
    ((5, 40, 7, 9, 200, 1, 1, 1, 0, 0), K1),           # C not a multiple of 32, K ragged against every tile
    ((1, 32, 6, 6, 16, 3, 3, 1, 1, 0), TC),            # one image, padding on all sides
    ((3, 64, 13, 13, 80, 3, 3, 1, 1, 1), TC),          # tiles straddle rows and images
    ((2, 96, 27, 27, 72, 5, 5, 1, 2, 1), TC),          # conv2-like
    ((2, 20, 15, 17, 24, 3, 5, 2, 1, 0), TC),          # stride 2, R != S, C padded
    ((1, 36, 23, 23, 40, 11, 11, 4, 0, 1), TC),        # conv1-like window and stride
    ((2, 32, 9, 9, 16, 2, 2, 1, 0, 1), TC),            # even window, no padding
    ((1, 32, 5, 5, 16, 3, 3, 1, 3, 0), TC),            # pad >= window: border outputs are pure bias
    ((2, 33, 10, 12, 300, 3, 3, 3, 2, 1), TC),         # stride 3, floor in the output extent
]


@pytest.mark.parametrize("shape,variant", EXACT_CASES)
def test_exact_on_small_integers(shape, variant):
    x, w, b = _int_tensors(shape, 500)
    got, desc = run_planned(shape, x, w, b, variant=variant)
    ref = oracle_out(shape, x, w, b)
    assert np.abs(ref).max() < 2 ** 24
    np.testing.assert_array_equal(got.astype(np.float64), ref, err_msg=desc)


@pytest.mark.parametrize("tile", range(5))
@pytest.mark.parametrize("split", [1, 2, 3, 8])
def test_every_tile_and_split_exact(tile, split):
    shape = (3, 64, 13, 13, 272, 3, 3, 1, 1, 1)
    x, w, b = _int_tensors(shape, 600)
    got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile, split_k=split)
    import re
    eff = int(re.search(r"split_k=(\d+)", desc).group(1))      # splits that would be empty are dropped
    assert f"id {tile}" in desc and (eff == split or (split == 8 and eff == 6))
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_k1conv_is_the_matrix_product():
    # Section 5 of the paper: for kernel size 1 the per-image im2col is the identity
    shape = (2, 64, 6, 5, 32, 1, 1, 1, 0, 0)
    x, w, _ = _int_tensors(shape, 700)
    got, _ = run_planned(shape, x, w, None, variant=K1)
    for n in range(2):
        ref = w.reshape(32, 64).astype(np.float64) @ x[n].reshape(64, 30).astype(np.float64)
        np.testing.assert_array_equal(got[n].reshape(32, 30).astype(np.float64), ref)


@pytest.mark.parametrize("shape,variant", [
    ((5, 480, 14, 14, 192, 1, 1, 1, 0, 1), K1),
    ((4, 256, 13, 13, 384, 3, 3, 1, 1, 1), TC),
    ((2, 96, 27, 27, 256, 5, 5, 1, 2, 1), TC),
    ((3, 50, 20, 20, 70, 3, 3, 2, 1, 0), TC),
])
def test_tf32_tolerance_on_real_values(shape, variant):
    x, w, b = _real_tensors(shape, 800)
    ref = oracle_out(shape, x, w, b)
    for bind in (False, True):
        got, desc = run_planned(shape, x, w, b, variant=variant, bind=bind)
        err = assert_parity(got, ref, TF32_TOL, desc)
        assert err > 1e-7      # it really ran in reduced precision (an fp32 path would be ~1e-7)


@pytest.mark.parametrize("cfg", [3, 4])
def test_baseline_configs_tf32(cfg):
    c = wl.CONFIGS[cfg]
    x, w, b = c.tensors()
    got, desc = run_planned(c.shape.as_tuple(), x, w, b)
    assert ("k1conv" if cfg == 3 else "tconv") in desc
    assert_parity(got, oracle_out(c.shape.as_tuple(), x, w, b), TF32_TOL, f"cfg{cfg} {desc}")


def test_same_result_twice_bitwise_and_tuned_plan():
    shape = (4, 128, 13, 13, 200, 3, 3, 1, 1, 1)
    x, w, b = _real_tensors(shape, 900)
    a, _ = run_planned(shape, x, w, b, variant=TC, split_k=3)
    c, _ = run_planned(shape, x, w, b, variant=TC, split_k=3)
    np.testing.assert_array_equal(a, c)          # split reduction is summed in split order: deterministic
    t, desc = run_planned(shape, x, w, b, tune=1)
    assert_parity(t, oracle_out(shape, x, w, b), TF32_TOL, desc)


# ---------------------------------------------------------------- halo (input-reuse) tconv kernel, tile ids 5..12
HALO_SHAPES = [
    (1, 32, 6, 6, 16, 3, 3, 1, 1, 0),            # one tile
    (3, 64, 13, 13, 80, 3, 3, 1, 1, 1),          # conv3-like, images share their zero rows
    (2, 96, 27, 27, 72, 5, 5, 1, 2, 1),          # conv2-like: slab of 248 / 376 rows
    (2, 40, 12, 10, 24, 3, 3, 1, 0, 0),          # no padding: outputs narrower than the row pitch
    (2, 32, 9, 11, 40, 2, 4, 1, 1, 1),           # R != S, even sizes
    (1, 48, 57, 57, 96, 3, 3, 1, 0, 1),          # space-to-depth view of an 11x11 stride-4 layer
    (2, 33, 8, 8, 300, 3, 3, 1, 2, 1),           # pad = window - 1: output larger than the input
]


@pytest.mark.parametrize("tile", [5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15])
@pytest.mark.parametrize("shape", HALO_SHAPES)
def test_halo_tiles_exact(shape, tile):
    x, w, b = _int_tensors(shape, 1100)
    got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile)
    assert "halo" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


@pytest.mark.parametrize("tile,split", [(6, 2), (7, 3), (10, 2), (11, 4), (12, 8), (9, 6)])
def test_halo_split_exact(tile, split):
    shape = (3, 96, 13, 13, 272, 3, 3, 1, 1, 1)
    x, w, b = _int_tensors(shape, 1200)
    got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile, split_k=split)
    assert "halo" in desc and "split_k=1 " not in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_halo_refused_where_it_does_not_apply():
    from paper_1606_00094_b200 import binding as B
    for shape in [(2, 32, 15, 17, 24, 3, 3, 2, 1, 0), (1, 32, 5, 5, 16, 3, 3, 1, 3, 0), (1, 32, 8, 8, 16, 1, 1, 1, 0, 0)]:
        with pytest.raises(B.BodaError) as e:
            B.ConvPlan(shape, variant=TC if shape[5] > 1 else K1, tile_id=6, s2d=0)
        assert e.value.status == B.BODA_ERR_UNSUPPORTED


# ---------------------------------------------------------------- space-to-depth view of strided layers
S2D_SHAPES = [
    (1, 3, 43, 43, 24, 11, 11, 4, 0, 1),         # AlexNet conv1-like: 11x11 stride 4 on 3 channels -> 3x3 on 48
    (2, 3, 227, 227, 96, 11, 11, 4, 0, 1),       # the real conv1 shape at batch 2
    (2, 20, 15, 17, 24, 3, 5, 2, 1, 0),          # stride 2 with padding, R != S
    (2, 8, 16, 16, 40, 2, 2, 2, 0, 1),           # window = stride: the view is a 1x1 convolution
    (1, 5, 20, 23, 33, 7, 7, 3, 3, 0),           # stride 3, window not a multiple of the stride, padding
    (3, 16, 9, 9, 16, 3, 3, 2, 1, 1),
    (2, 3, 50, 61, 16, 7, 7, 4, 3, 1),           # stride 4 on 3 channels with padding and odd extents (the specialised staging kernel)
    (1, 3, 300, 251, 16, 9, 9, 4, 2, 0),         # rows longer than 256 staged columns: more than one pass of staging loads
]


@pytest.mark.parametrize("shape", S2D_SHAPES)
@pytest.mark.parametrize("tile", [-1, 1, 6, 10])
def test_space_to_depth_exact(shape, tile):
    x, w, b = _int_tensors(shape, 1300)
    try:
        got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile, s2d=1)
    except Exception as e:                       # a halo tile is refused when the view has a single tap
        from paper_1606_00094_b200 import binding as B
        assert isinstance(e, B.BodaError) and e.status == B.BODA_ERR_UNSUPPORTED and tile in (6, 10) and shape[5] <= shape[7]
        return
    assert "s2d" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


# ---- the first-layer kernel (tiles 23..25): 3 channels, stride 4, no padding, read straight from NCHW by bulk copies
# and re-laid-out in shared memory (second channel chunk as 64-byte rows)
FIRST_SHAPES = [
    (1, 3, 227, 227, 96, 11, 11, 4, 0, 1),       # configuration 2: the tensor's last floats are not a whole 16-byte piece
    (3, 3, 227, 227, 96, 11, 11, 4, 0, 1),       # images start at odd float offsets
    (2, 3, 67, 67, 80, 11, 11, 4, 0, 0),         # one tile per image, K ragged against every tile, no ReLU
    (4, 3, 99, 83, 40, 9, 11, 4, 0, 1),          # R != S, non-square image, several tiles per image
    (2, 3, 61, 50, 24, 7, 5, 4, 0, 1),           # 2 x 2 block taps
    (5, 3, 35, 35, 16, 8, 8, 4, 0, 1),           # window a multiple of the stride; tiny output (7 x 7)
    (1, 3, 131, 259, 32, 11, 11, 4, 0, 1),       # wide rows
]


@pytest.mark.parametrize("shape", FIRST_SHAPES)
@pytest.mark.parametrize("tile", [23, 24, 25])
def test_first_layer_kernel_exact(shape, tile):
    x, w, b = _int_tensors(shape, 1350)
    got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile)
    assert "first_512x" in desc and f"id {tile}" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_first_layer_kernel_real_values_bound_filters_and_refusals():
    from paper_1606_00094_b200 import binding as B
    shape = (2, 3, 227, 227, 96, 11, 11, 4, 0, 1)
    x, w, b = _real_tensors(shape, 1360)
    ref = oracle_out(shape, x, w, b)
    for bind in (False, True):
        got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=24, bind=bind)
        assert_parity(got, ref, TF32_TOL, desc)
    for bad in [(2, 4, 67, 67, 32, 11, 11, 4, 0, 1),      # 4 channels
                (2, 3, 67, 67, 32, 11, 11, 2, 0, 1),      # stride 2
                (2, 3, 67, 67, 32, 11, 11, 4, 1, 1),      # padding
                (2, 3, 67, 67, 32, 13, 13, 4, 0, 1)]:     # 4 x 4 block taps
        with pytest.raises(B.BodaError):
            B.ConvPlan(bad, variant=TC, tile_id=24)


def test_space_to_depth_off_and_auto_agree_with_oracle():
    shape = (2, 3, 99, 99, 96, 11, 11, 4, 0, 1)
    x, w, b = _real_tensors(shape, 1400)
    ref = oracle_out(shape, x, w, b)
    a, da = run_planned(shape, x, w, b, variant=TC, s2d=0)
    c, dc = run_planned(shape, x, w, b)                      # automatic: tconv through the space-to-depth view
    assert "s2d" not in da and "tconv" in dc and ("s2d" in dc or "gconv" in dc)     # automatic: the view or the gather kernel
    assert_parity(a, ref, TF32_TOL, da)
    assert_parity(c, ref, TF32_TOL, dc)


def test_space_to_depth_refused_for_stride_one():
    from paper_1606_00094_b200 import binding as B
    with pytest.raises(B.BodaError) as e:
        B.ConvPlan((1, 32, 8, 8, 16, 3, 3, 1, 1, 0), variant=TC, s2d=1)
    assert e.value.status == B.BODA_ERR_UNSUPPORTED


# ---- gather kernel (tiles 16..19): the input tile is built by producer warps straight from NCHW
GATHER_CASES = [
    (2, 3, 23, 23, 40, 11, 11, 4, 0, 1),       # conv1-like: no padding, 363 reduction indices (ragged last chunk)
    (1, 3, 32, 32, 16, 3, 3, 1, 1, 1),         # configuration 1: one ragged chunk, padding on all sides
    (3, 8, 15, 17, 24, 3, 5, 2, 1, 0),         # stride 2, R != S
    (2, 16, 9, 9, 130, 5, 5, 1, 2, 1),         # several channel tiles per pixel tile, 400 indices
    (1, 4, 6, 6, 16, 3, 3, 1, 3, 0),           # pad >= window: border outputs are pure bias
    (7, 3, 40, 40, 96, 7, 7, 2, 3, 1),         # more tiles than one wave of CTAs would need at batch 7? (2800 points)
    (1, 32, 8, 8, 16, 2, 2, 1, 0, 1),          # exactly four full chunks, no tail
]


@pytest.mark.parametrize("shape", GATHER_CASES)
@pytest.mark.parametrize("tile", [16, 17, 18, 19])
def test_gather_tiles_exact(shape, tile):
    x, w, b = _int_tensors(shape, 2100)
    got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile)
    assert "gconv" in desc and f"id {tile}" in desc
    ref = oracle_out(shape, x, w, b)
    assert np.abs(ref).max() < 2 ** 24
    np.testing.assert_array_equal(got.astype(np.float64), ref, err_msg=desc)


def test_gather_conv1_shape_real_values_and_persistence():
    # 60 500 output points at batch 20 = 473 tiles on 148 persistent CTAs: several tiles per CTA, ragged last tile
    shape = (20, 3, 227, 227, 96, 11, 11, 4, 0, 1)
    x = wl.uniform(2200, (20, 3, 227, 227), 0.0, 1.0)
    w = wl.normal(2201, (96, 3, 11, 11), 0, (2.0 / 363) ** 0.5)
    b = wl.normal(2202, (96,), 0, 0.01)
    ref = oracle_out(shape, x, w, b)
    for tile, bind in ((17, False), (17, True), (16, True), (18, True)):
        got, desc = run_planned(shape, x, w, b, variant=TC, tile_id=tile, bind=bind)
        assert "gconv" in desc
        assert_parity(got, ref, TF32_TOL, desc)
    a, _ = run_planned(shape, x, w, b, variant=TC, tile_id=17, bind=True)
    a2, _ = run_planned(shape, x, w, b, variant=TC, tile_id=17, bind=True)
    assert np.array_equal(a, a2)                # the same plan twice: bit for bit


def test_gather_refused_where_it_does_not_apply():
    from paper_1606_00094_b200 import binding as B
    with pytest.raises(B.BodaError):
        B.ConvPlan((1, 256, 13, 13, 64, 3, 3, 1, 1, 1), variant=TC, tile_id=17)        # 2304 reduction indices: table too small
    with pytest.raises(B.BodaError):
        B.ConvPlan((1, 3, 32, 32, 16, 3, 3, 1, 1, 1), variant=TC, tile_id=17, split_k=2)
    with pytest.raises(B.BodaError):
        B.ConvPlan((1, 3, 33, 33, 16, 3, 3, 2, 1, 1), variant=TC, tile_id=17, s2d=1)


# the gather kernel also runs 1x1 layers straight from NCHW (consecutive output points are consecutive addresses):
# no staged copy of the input, which is what large batches of such layers spend their time on otherwise
@pytest.mark.parametrize("shape", [
    (5, 40, 7, 9, 200, 1, 1, 1, 0, 0),            # C not a multiple of 32, K ragged against every tile, tiles straddle images
    (3, 480, 14, 14, 192, 1, 1, 1, 0, 1),         # configuration 3's layer
    (2, 64, 9, 9, 24, 1, 1, 2, 0, 1),             # stride 2
])
@pytest.mark.parametrize("tile", [16, 19])
def test_gather_tiles_run_k1conv_exact(shape, tile):
    x, w, b = _int_tensors(shape, 1700)
    got, desc = run_planned(shape, x, w, b, variant=K1, tile_id=tile)
    assert "gconv" in desc and "k1conv" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_1x1_layers_avoid_the_staged_copy_at_every_batch():
    # rows TMA can address (H*W a multiple of 4): the NCHW kernel; otherwise the gather kernel once the batch is large
    from paper_1606_00094_b200 import binding as B
    big = B.ConvPlan((256, 480, 14, 14, 192, 1, 1, 1, 0, 1))
    small = B.ConvPlan((5, 480, 14, 14, 192, 1, 1, 1, 0, 1))
    odd = B.ConvPlan((256, 480, 13, 13, 192, 1, 1, 1, 0, 1))
    try:
        assert "k1nchw_128x192" in big.describe() and "k1nchw" in small.describe()
        assert "gconv" in odd.describe()
    finally:
        big.close(); small.close(); odd.close()


# ---- 1x1 layers by TMA straight from NCHW (tiles 20..22): the input tile is an MN-major tensor-core operand
K1N_SHAPES = [
    (2, 64, 14, 14, 48, 1, 1, 1, 0, 1),           # two tiles per image, the second ragged (196 = 128 + 68)
    (5, 40, 6, 6, 200, 1, 1, 1, 0, 0),            # image smaller than a tile, C not a multiple of 32, K ragged against every tile
    (3, 480, 14, 14, 192, 1, 1, 1, 0, 1),         # configuration 3's layer
    (1, 32, 16, 24, 16, 1, 1, 1, 0, 1),           # exactly three tiles, one reduction step
]


@pytest.mark.parametrize("shape", K1N_SHAPES)
@pytest.mark.parametrize("tile", [20, 21, 22])
@pytest.mark.parametrize("split", [0, 2, 4])          # 0: the cost model's choice; otherwise a cluster of that many CTAs per tile
def test_k1conv_from_nchw_exact(shape, tile, split):
    x, w, b = _int_tensors(shape, 1800)
    got, desc = run_planned(shape, x, w, b, variant=K1, tile_id=tile, split_k=split)
    assert "k1nchw_128x" in desc and f"id {tile}" in desc
    if split and shape[1] >= 32 * split:
        assert f"split_k={split}" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_k1conv_from_nchw_split_runs_twice_bitwise_equal():
    """The cluster sum adds the partial accumulators in rank order: two runs must agree bit for bit."""
    shape = (5, 480, 14, 14, 192, 1, 1, 1, 0, 1)
    x, w, b = _real_tensors(shape, 1850)
    a, desc = run_planned(shape, x, w, b, variant=K1, tile_id=20, split_k=4)
    c, _ = run_planned(shape, x, w, b, variant=K1, tile_id=20, split_k=4)
    assert "split_k=4" in desc
    np.testing.assert_array_equal(a, c)
    assert_parity(a, oracle_out(shape, x, w, b), TF32_TOL, desc)


def test_k1conv_from_nchw_on_real_values_is_the_choice_for_configuration_3_and_refuses_what_it_cannot_address():
    from paper_1606_00094_b200 import binding as B
    c = wl.CONFIGS[3]
    x, w, b = c.tensors()
    got, desc = run_planned(c.shape.as_tuple(), x, w, b)
    assert "k1nchw" in desc           # one kernel, no staging: faster than staging + the tiled kernel at this size
    # the input is used as it lies in memory: the tensor core truncates it to TF32 (no rounding pass), still inside the bar
    assert_parity(got, oracle_out(c.shape.as_tuple(), x, w, b), TF32_TOL, desc)
    with pytest.raises(B.BodaError):
        B.ConvPlan((2, 64, 7, 9, 32, 1, 1, 1, 0, 1), variant=K1, tile_id=20)          # rows of 63 floats: not a multiple of 16 bytes
    with pytest.raises(B.BodaError):
        B.ConvPlan((2, 64, 8, 8, 32, 1, 1, 2, 0, 1), variant=K1, tile_id=20)          # stride 2
    auto = B.ConvPlan((2, 64, 7, 9, 32, 1, 1, 1, 0, 1), variant=K1)                   # automatic selection falls back to the staged path
    try:
        assert "k1nchw" not in auto.describe()
    finally:
        auto.close()


def test_tuned_choice_is_remembered_in_the_cache_file(tmp_path, monkeypatch):
    import time
    from paper_1606_00094_b200 import binding as B
    cache = tmp_path / "tune.txt"
    monkeypatch.setenv("BODA_TUNE_CACHE", str(cache))
    shape = (2, 64, 12, 12, 96, 3, 3, 1, 1, 1)
    t0 = time.time(); first = B.ConvPlan(shape, tune=1); t_first = time.time() - t0
    t0 = time.time(); second = B.ConvPlan(shape, tune=1); t_second = time.time() - t0
    try:
        lines = cache.read_text().strip().splitlines()
        assert len(lines) == 1 and lines[0].startswith("t4:2,64,12,12,96,3,3,1,1,")       # one entry, keyed by tile-table version and shape
        assert second.describe() == first.describe()
        assert t_second < t_first                                                          # no candidates were timed again
        # an entry written for other tile tables is ignored, not misread
        cache.write_text(lines[0].replace("t4:", "t2:", 1) + "\n")
        third = B.ConvPlan(shape, tune=1)
        third.close()
        assert len(cache.read_text().strip().splitlines()) == 2
    finally:
        first.close(); second.close()


def test_workspace_limit_steers_the_plan():
    """opts.max_workspace: tiles whose staged input does not fit are not considered; automatic selection then lands on
    a kernel that stages nothing (or the FP32 kernel), a forced tile that needs more is refused with BODA_ERR_NOMEM."""
    from paper_1606_00094_b200 import binding as B
    shape = (4, 64, 13, 13, 96, 3, 3, 1, 1, 1)
    x, w, b = _real_tensors(shape, 3100)
    ref = oracle_out(shape, x, w, b)
    free = B.ConvPlan(shape)
    need = B.boda_conv_plan_workspace_bytes(free.handle)
    free.close()
    assert need > 0                                           # the unconstrained choice stages its input
    roomy = B.ConvPlan(shape, max_workspace=need)
    assert B.boda_conv_plan_workspace_bytes(roomy.handle) <= need
    roomy.close()
    tight = B.ConvPlan(shape, max_workspace=1024)
    try:
        assert B.boda_conv_plan_workspace_bytes(tight.handle) <= 1024, tight.describe()
        import torch
        got = tight(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda()).cpu().numpy()
        assert_parity(got, ref, TF32_TOL, tight.describe())
    finally:
        tight.close()
    with pytest.raises(B.BodaError) as e:
        B.ConvPlan(shape, variant=TC, tile_id=2, max_workspace=1024)
    assert e.value.status == B.BODA_ERR_NOMEM
