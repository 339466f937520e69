"""GPU parity of the FP32 CUDA-core path (DIRECT) and of max-pooling against the fp64 oracle."""
import numpy as np
import pytest

from oracle import conv_oracle as orc
from paper_1606_00094_b200 import workloads as wl
from helpers import FP32_TOL, assert_parity, oracle_out, run_planned

pytestmark = pytest.mark.gpu

# (N,C,H,W,K,R,S,stride,pad,relu): tiny, ragged in every tile dimension, several tiles, odd strides
SHAPES = [
    (1, 1, 3, 3, 1, 2, 2, 1, 0, 0),
    (1, 3, 32, 32, 16, 3, 3, 1, 1, 1),
    (2, 3, 7, 9, 4, 3, 3, 1, 1, 0),
    (1, 5, 11, 8, 3, 5, 3, 2, 2, 1),
    (3, 2, 37, 41, 19, 2, 2, 1, 0, 1),
    (2, 7, 23, 23, 33, 11, 11, 4, 0, 1),
    (1, 130, 9, 9, 70, 1, 1, 1, 0, 1),
    (2, 6, 5, 5, 140, 3, 3, 1, 3, 0),      # pad >= window: border outputs are pure bias
    (1, 2, 9, 7, 3, 4, 2, 3, 1, 1),
    (5, 16, 14, 14, 24, 1, 1, 1, 0, 1),
]


def _tensors(shape, seed):
    N, C, H, W, K, R, S, st, pad, relu = shape
    return (wl.normal(seed, (N, C, H, W)), wl.normal(seed + 1, (K, C, R, S), 0, 0.2), wl.normal(seed + 2, (K,), 0, 0.1))


@pytest.mark.parametrize("shape", SHAPES)
def test_direct_matches_oracle(shape):
    x, w, b = _tensors(shape, 1000)
    got, desc = run_planned(shape, x, w, b, variant=0, math=1)
    assert "variant=direct" in desc
    assert_parity(got, oracle_out(shape, x, w, b), FP32_TOL, desc)


@pytest.mark.parametrize("tile", range(12))        # 0..8: GEMM-blocked tiles; 9..11: pixel-per-thread tiles
def test_every_direct_tile(tile):
    shape = (2, 5, 19, 17, 37, 3, 3, 2, 1, 1)
    x, w, b = _tensors(shape, 2000)
    got, desc = run_planned(shape, x, w, b, variant=0, math=1, tile_id=tile)
    assert f"id {tile}" in desc
    assert_parity(got, oracle_out(shape, x, w, b), FP32_TOL, desc)


def test_direct_is_exact_on_small_integers():
    # integer inputs in [-8, 8]: every product and partial sum is exact in fp32, so any indexing slip shows
    shape = (2, 6, 12, 13, 20, 3, 5, 2, 2, 0)
    N, C, H, W, K, R, S, st, pad, relu = shape
    x, w, b = wl.integers(1, (N, C, H, W)), wl.integers(2, (K, C, R, S)), wl.integers(3, (K,))
    got, _ = run_planned(shape, x, w, b, variant=0, math=1)
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b))


def test_no_bias_and_no_relu():
    shape = (1, 4, 10, 10, 8, 3, 3, 1, 1, 0)
    x, w, _ = _tensors(shape, 3000)
    got, _ = run_planned(shape, x, w, None, variant=0, math=1)
    ref = oracle_out(shape, x, w, None)
    assert (ref < 0).any()
    assert_parity(got, ref, FP32_TOL)


@pytest.mark.parametrize("cfg", [1, 2])
def test_baseline_configs_fp32(cfg):
    c = wl.CONFIGS[cfg]
    x, w, b = c.tensors()
    got, desc = run_planned(c.shape.as_tuple(), x, w, b, math=1)
    assert_parity(got, oracle_out(c.shape.as_tuple(), x, w, b), FP32_TOL, f"cfg{cfg} {desc}")


def test_one_call_entry_point_and_host_entry_point():
    import torch
    from paper_1606_00094_b200 import binding as B
    shape = (2, 3, 15, 15, 10, 5, 5, 2, 2, 1)
    N, C, H, W, K, R, S, st, pad, relu = shape
    x, w, b = _tensors(shape, 4000)
    ref = oracle_out(shape, x, w, b)
    out = B.conv_fwd(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda(), st, pad, True)
    torch.cuda.synchronize()
    tol = 5e-3   # automatic math may choose TF32
    assert_parity(out.cpu().numpy(), ref, tol)
    hx, hw, hb = (torch.from_numpy(t).pin_memory() for t in (x, w, b))
    ho = torch.empty(ref.shape, dtype=torch.float32).pin_memory()
    for _ in range(2):
        ho.fill_(float("nan"))
        B.boda_conv_fwd_host(hx, hw, hb, ho, N, C, H, W, K, R, S, st, pad, relu)
        assert_parity(ho.numpy(), ref, tol)
    B.boda_clear_caches()


def test_maxpool_matches_oracle_exactly():
    import torch
    from paper_1606_00094_b200 import binding as B
    for (N, C, H, W) in [(1, 1, 5, 5), (2, 3, 13, 14), (3, 5, 27, 27), (2, 4, 55, 55)]:
        x = wl.normal(7, (N, C, H, W))
        got = B.maxpool_fwd(torch.from_numpy(x).cuda()).cpu().numpy()
        np.testing.assert_array_equal(got.astype(np.float64), orc.maxpool_fwd(x))


def test_forced_illegal_variant_is_refused():
    from paper_1606_00094_b200 import binding as B
    with pytest.raises(B.BodaError) as e:
        B.boda_conv_plan_create((1, 3, 8, 8, 4, 3, 3, 1, 1, 1), _opts(B, variant=B.BODA_VARIANT_K1CONV))
    assert e.value.status == B.BODA_ERR_UNSUPPORTED
    with pytest.raises(B.BodaError) as e:
        B.boda_conv_plan_create((1, 3, 8, 8, 4, 3, 3, 1, 1, 1), _opts(B, variant=0, tile_id=99))
    assert e.value.status == B.BODA_ERR_UNSUPPORTED


def _opts(B, **kw):
    o = B.boda_plan_opts_default()
    for k, v in kw.items():
        setattr(o, k, v)
    return o


# ---- pixel-per-thread tiles (small input-channel count): exact on integers, every shape quirk
PIXEL_CASES = [
    (1, 3, 32, 32, 16, 3, 3, 1, 1, 1),          # configuration 1
    (3, 3, 45, 70, 20, 5, 5, 2, 2, 1),          # patch edges on both sides, stride 2, ragged channel group
    (2, 3, 59, 59, 40, 11, 11, 4, 0, 1),        # conv1-like window and stride
    (2, 1, 9, 40, 5, 3, 3, 1, 1, 0),            # one input channel, fewer outputs than a group
    (1, 4, 7, 7, 70, 7, 7, 1, 3, 1),            # window as large as the image, three channel groups
    (5, 2, 33, 65, 9, 2, 4, 3, 0, 0),           # R != S, stride 3, floor in the output extent
]


@pytest.mark.parametrize("shape", PIXEL_CASES)
@pytest.mark.parametrize("tile", [9, 10, 11])
def test_pixel_tiles_exact(shape, tile):
    N, C, H, W, K, R, S, st, pad, relu = shape
    x, w, b = wl.integers(4100, (N, C, H, W)), wl.integers(4101, (K, C, R, S)), wl.integers(4102, (K,))
    got, desc = run_planned(shape, x, w, b, variant=0, math=1, tile_id=tile)
    assert "direct_pixel" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)


def test_pixel_tile_is_the_automatic_choice_for_large_batches_of_configuration_1_and_meets_the_fp32_bar():
    shape = (40, 3, 32, 32, 16, 3, 3, 1, 1, 1)          # configuration 1's layer at batch 40: 40 960 output pixels
    x, w, b = _tensors(shape, 4200)
    got, desc = run_planned(shape, x, w, b, math=1)
    assert "direct_rtc_k16" in desc or "direct_pixel_k16" in desc      # the run-time compiled form where NVRTC is there
    assert_parity(got, oracle_out(shape, x, w, b), FP32_TOL, desc)
    c = wl.CONFIGS[1]                                    # at batch 1 the blocked tiles stay the choice
    x, w, b = c.tensors()
    got, desc = run_planned(c.shape.as_tuple(), x, w, b, math=1)
    assert "direct_pixel" not in desc          # (the run-time compiled tile where NVRTC is there, else a blocked tile)
    assert_parity(got, oracle_out(c.shape.as_tuple(), x, w, b), FP32_TOL, desc)


def test_pixel_tile_refused_when_the_patch_does_not_fit():
    from paper_1606_00094_b200 import binding as B
    with pytest.raises(B.BodaError):
        B.ConvPlan((1, 64, 56, 56, 32, 11, 11, 4, 0, 1), variant=0, math=1, tile_id=11)


# ---- tiles compiled at run time for the exact shape (Section 4 of the paper): ids 12..15
def _rtc_or_skip():
    from paper_1606_00094_b200 import binding as B
    try:
        B.boda_direct_rtc_compile((1, 3, 8, 8, 4, 3, 3, 1, 1, 0), 4)
    except B.BodaError as e:
        if e.status == B.BODA_ERR_UNSUPPORTED:
            pytest.skip("NVRTC is not available on this machine")
        raise


@pytest.mark.parametrize("shape", PIXEL_CASES)
@pytest.mark.parametrize("tile", [12, 13, 14, 15])
def test_rtc_tiles_exact(shape, tile):
    _rtc_or_skip()
    from paper_1606_00094_b200 import binding as B
    N, C, H, W, K, R, S, st, pad, relu = shape
    x, w, b = wl.integers(4300, (N, C, H, W)), wl.integers(4301, (K, C, R, S)), wl.integers(4302, (K,))
    try:
        B.boda_direct_rtc_compile(shape, (4, 8, 16, 32)[tile - 12])
    except B.BodaError as e:          # filters and patch beyond 48 KB of shared memory: the plan is refused as well
        assert e.status == B.BODA_ERR_UNSUPPORTED
        with pytest.raises(B.BodaError):
            B.ConvPlan(shape, variant=0, math=1, tile_id=tile)
        return
    got, desc = run_planned(shape, x, w, b, variant=0, math=1, tile_id=tile)
    assert "direct_rtc" in desc and "rtc block=" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)
    got2, _ = run_planned(shape, x, w, None, variant=0, math=1, tile_id=tile)          # no bias
    np.testing.assert_array_equal(got2.astype(np.float64), oracle_out(shape, x, w, None))


def test_rtc_tile_on_real_values_and_refusals():
    _rtc_or_skip()
    from paper_1606_00094_b200 import binding as B
    shape = (6, 3, 64, 48, 24, 7, 7, 2, 3, 1)
    x, w, b = _tensors(shape, 4400)
    got, desc = run_planned(shape, x, w, b, variant=0, math=1, tile_id=13)
    assert_parity(got, oracle_out(shape, x, w, b), FP32_TOL, desc)
    with pytest.raises(B.BodaError):                      # 256 channels of 3x3: the filters alone exceed shared memory
        B.ConvPlan((1, 256, 13, 13, 64, 3, 3, 1, 1, 1), variant=0, math=1, tile_id=14)


@pytest.mark.parametrize("rows", ["2", "4"])
def test_rtc_tile_with_several_rows_per_thread(rows, monkeypatch):
    _rtc_or_skip()
    monkeypatch.setenv("BODA_RTC_ROWS_PER_THREAD", rows)        # large layers choose this themselves; forced here on a small one
    shape = (3, 3, 45, 70, 20, 5, 5, 2, 2, 1)
    N, C, H, W, K, R, S, st, pad, relu = shape
    x, w, b = wl.integers(4500, (N, C, H, W)), wl.integers(4501, (K, C, R, S)), wl.integers(4502, (K,))
    got, desc = run_planned(shape, x, w, b, variant=0, math=1, tile_id=13)
    assert f"rows={rows}" in desc
    np.testing.assert_array_equal(got.astype(np.float64), oracle_out(shape, x, w, b), err_msg=desc)
