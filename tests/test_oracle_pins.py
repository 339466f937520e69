"""Pins of the fp64 CPU oracle against facts it did not produce itself.

Each test ties ``oracle/conv_oracle.c`` to something the paper or the mathematics fixes: the
numbers of the paper's worked example, hand-computed outputs, closed forms, identities with a
plain matrix product / a shift / an explicitly padded or sub-sampled problem, a brute-force
im2col + matmul written here with numpy index arithmetic, and two library routines.
"""
import math
import os

import numpy as np
import pytest

from oracle import conv_oracle as orc
from paper_1606_00094_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kv(path):
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, v = [t.strip() for t in line.split("=")]
            out[k] = float(v)
    return out


# ---------------------------------------------------------------- paper's worked example (Sec. 2, 3)
def test_worked_example_shapes_and_counts():
    g = _kv(os.path.join(GOLDEN, "paper_worked_example.txt"))
    H, W, C, K, R = int(g["in_Y"]), int(g["in_X"]), int(g["IC"]), int(g["OC"]), int(g["KSZ"])
    st, pad = int(g["stride"]), int(g["pad"])
    P = orc.conv_out_dim(H, R, st, pad)
    Q = orc.conv_out_dim(W, R, st, pad)
    assert (P, Q) == (g["out_Y"], g["out_X"])
    assert P * Q * K == g["output_points"]
    assert P * Q == g["input_slices"] and K == g["filter_slices"]
    assert R * R * C == g["slice_elems"]
    assert orc.conv_macs(1, C, H, W, K, R, R, st, pad) == g["macs"]
    assert 4 * P * Q * K == g["outmat_bytes"]
    assert 4 * P * Q * R * R * C == g["inmat_bytes"]
    assert 4 * R * R * C * K == g["filtsmat_bytes"]
    total = g["outmat_bytes"] + g["inmat_bytes"] + g["filtsmat_bytes"]
    assert round(g["macs"] / total, 1) == g["ai_printed"]
    # the oracle really produces an output of that shape on that input shape
    x = wl.uniform(1, (1, C, 21, 21), -1, 1)            # same R/stride on a small image
    f = wl.normal(2, (K, C, R, R))
    assert orc.conv_fwd(x, f, stride=st).shape == (1, K, 8, 8)


def test_min_bytes_counts_each_tensor_once():
    # The worked example (205x205x3 input, 96 7x7 filters, stride 2).  The paper's AI figure prints 3.84 MB for the
    # output and 56 448 B for the filters; the input itself is 205*205*3 floats = 504 300 B (counted by hand: the
    # figure counts the im2col matrix instead) and the bias 96 floats = 384 B.
    assert orc.conv_min_bytes(1, 3, 205, 205, 96, 7, 7, 2, 0) == 3840000 + 56448 + 504300 + 384
    # a second hand count: 1x1x1x1 input, one 1x1 filter -> 4 tensors of one float each
    assert orc.conv_min_bytes(1, 1, 1, 1, 1, 1, 1, 1, 0) == 16


def test_sgemm_ai_matches_table1():
    for line in open(os.path.join(GOLDEN, "sgemm_table1.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        n, nbytes, flops, ai = [float(t) for t in line.split()]
        n = int(n)
        assert abs(4 * 3 * n * n - nbytes) / nbytes < 5e-3          # printed to 3 digits
        assert abs(2 * n ** 3 - flops) / flops < 5e-3
        assert abs(orc.sgemm_ai(n, n, n) - ai) / ai < 5e-3
    # non-square: 2MNK / 4(MN+MK+KN), Section 4
    assert orc.sgemm_ai(10000, 96, 147) == pytest.approx(2 * 10000 * 96 * 147 / (4 * (10000 * 96 + 10000 * 147 + 147 * 96)))


# ---------------------------------------------------------------- hand-computed cases
def _rows(txt):
    return np.array([[float(v) for v in row.split()] for row in txt.split("/")])


def test_hand_cases_from_fixture():
    # Derivations (in = [[1,2,3],[4,5,6],[7,8,9]]):
    #  i   filt [[1,2],[3,4]]: out[0,0] = 1*1+2*2+4*3+5*4 = 37, out[0,1] = 2+6+15+24 = 47,
    #      out[1,0] = 4+10+21+32 = 67, out[1,1] = 5+12+24+36 = 77.
    #  ii  stride 2, pad 1 (5x5 padded): out[0,0] sees only in[0,0] under filt[1,1] -> 4;
    #      out[0,1] = 2*3 + 3*4 = 18; out[1,0] = 4*2 + 7*4 = 36; out[1,1] = 5+12+24+36 = 77.
    #  iii filt [[1,0],[0,-1]]: in[y,x] - in[y+1,x+1] = -4, plus bias 0.5 -> -3.5; ReLU -> 0.
    #  iv  3x3 ones, pad 1: neighbourhood sums, e.g. corner 1+2+4+5 = 12, centre 45.
    x = np.arange(1, 10, dtype=np.float64).reshape(1, 1, 3, 3)
    n = 0
    for line in open(os.path.join(GOLDEN, "hand_cases.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        name, filt, stride, pad, bias, relu, exp = [t.strip() for t in line.split(";")]
        f = _rows(filt)[None, None]
        got = orc.conv_fwd(x, f, np.array([float(bias)]), stride=int(stride), pad=int(pad), relu=bool(int(relu)))
        np.testing.assert_array_equal(got[0, 0], _rows(exp), err_msg=name)
        n += 1
    assert n == 5


def test_two_channel_two_filter_hand_case():
    # in[c=0] = [[1,2],[3,4]], in[c=1] = [[10,20],[30,40]]; 1x1 filters k0 = (1, 0.1), k1 = (-1, 1).
    # k0: 1*in0 + 0.1*in1 = [[2,4],[6,8]]; k1: in1 - in0 = [[9,18],[27,36]].
    x = np.array([[[[1, 2], [3, 4]], [[10, 20], [30, 40]]]], dtype=np.float64)
    f = np.array([[[[1.0]], [[0.1]]], [[[-1.0]], [[1.0]]]])
    got = orc.conv_fwd(x, f)
    np.testing.assert_allclose(got[0, 0], [[2, 4], [6, 8]], rtol=1e-15)
    np.testing.assert_array_equal(got[0, 1], [[9, 18], [27, 36]])


def test_no_flip_and_rs_orientation():
    # A 1x3 filter (R=1, S=3) [1, 10, 100] over the row [1, 2, 3, 4]: cross-correlation gives
    # 1*1 + 2*10 + 3*100 = 321 and 2 + 30 + 400 = 432 (a flipped kernel would give 123, 234).
    x = np.array([1.0, 2, 3, 4]).reshape(1, 1, 1, 4)
    f = np.array([1.0, 10, 100]).reshape(1, 1, 1, 3)
    np.testing.assert_array_equal(orc.conv_fwd(x, f)[0, 0], [[321, 432]])
    # the transposed problem (R=3, S=1) on a column gives the same numbers down the column
    np.testing.assert_array_equal(orc.conv_fwd(x.reshape(1, 1, 4, 1), f.reshape(1, 1, 3, 1))[0, 0], [[321], [432]])


# ---------------------------------------------------------------- closed forms
def test_all_ones_counts_in_bounds_taps():
    C = 5
    x = np.ones((2, C, 4, 4))
    f = np.ones((3, C, 3, 3))
    got = orc.conv_fwd(x, f, pad=1)
    edge = np.array([[4, 6, 6, 4], [6, 9, 9, 6], [6, 9, 9, 6], [4, 6, 6, 4]], dtype=np.float64) * C
    for n in range(2):
        for k in range(3):
            np.testing.assert_array_equal(got[n, k], edge)


def test_pad_not_smaller_than_window_gives_pure_bias_border():
    x = wl.uniform(3, (1, 2, 3, 3), -1, 1)
    f = wl.normal(4, (2, 2, 2, 2))
    b = np.array([0.25, -0.5])
    got = orc.conv_fwd(x, f, b, pad=2)
    assert got.shape == (1, 2, 6, 6)
    np.testing.assert_array_equal(got[0, :, 0, :], np.repeat(b[:, None], 6, 1))   # first row: only padding


# ---------------------------------------------------------------- identities
SHAPES = [
    # N, C, H, W, K, R, S, stride, pad
    (2, 3, 7, 9, 4, 3, 3, 1, 1),
    (1, 5, 11, 8, 3, 5, 3, 2, 2),
    (3, 2, 6, 6, 5, 2, 2, 1, 0),
    (1, 4, 13, 13, 6, 3, 3, 2, 0),
    (2, 3, 23, 23, 7, 11, 11, 4, 0),
    (1, 6, 5, 5, 2, 1, 1, 1, 0),
    (1, 2, 9, 7, 3, 4, 2, 3, 1),
]


def _rand(shape, seed):
    N, C, H, W, K, R, S, st, pad = shape
    x = wl.normal(seed, (N, C, H, W)).astype(np.float64)
    f = wl.normal(seed + 1, (K, C, R, S)).astype(np.float64)
    b = wl.normal(seed + 2, (K,)).astype(np.float64)
    return x, f, b


def _im2col_matmul(x, f, b, stride, pad):
    """Brute force of Section 3: inmat (one row per output point, one column per (c,r,s)) times filtsmat."""
    N, C, H, W = x.shape
    K, _, R, S = f.shape
    xp = np.zeros((N, C, H + 2 * pad, W + 2 * pad))
    xp[:, :, pad:pad + H, pad:pad + W] = x
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    inmat = np.empty((N * P * Q, C * R * S))
    row = 0
    for n in range(N):
        for p in range(P):
            for q in range(Q):
                inmat[row] = xp[n, :, p * stride:p * stride + R, q * stride:q * stride + S].reshape(-1)
                row += 1
    filtsmat = f.reshape(K, -1).T                       # Section 3: filtsmat is filts reshaped to (C*R*S) x K
    outmat = inmat @ filtsmat + b[None, :]
    return outmat.reshape(N, P, Q, K).transpose(0, 3, 1, 2)


@pytest.mark.parametrize("shape", SHAPES)
def test_equals_im2col_matmul(shape):
    x, f, b = _rand(shape, 100)
    st, pad = shape[7], shape[8]
    ref = _im2col_matmul(x, f, b, st, pad)
    got = orc.conv_fwd(x, f, b, stride=st, pad=pad)
    assert got.shape == ref.shape
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.conv_fwd(x, f, b, stride=st, pad=pad, relu=True), np.maximum(ref, 0), rtol=1e-12, atol=1e-12)


def test_ksz1_is_a_matrix_product():
    # Section 5: for KSZ = 1 the per-image im2col is the identity, so out[n] = filt[KxC] @ in[n][Cx(HW)]
    x, f, b = _rand((3, 17, 6, 5, 9, 1, 1, 1, 0), 7)
    got = orc.conv_fwd(x, f, b)
    for n in range(3):
        ref = f.reshape(9, 17) @ x[n].reshape(17, 30) + b[:, None]
        np.testing.assert_allclose(got[n].reshape(9, 30), ref, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("pad", [0, 1, 2])
def test_delta_filter_is_a_shift(pad):
    C, H, W, R, S = 3, 6, 7, 3, 4
    x = wl.normal(11, (2, C, H, W)).astype(np.float64)
    for (c0, r0, s0) in [(0, 0, 0), (1, 2, 1), (2, 1, 3)]:
        f = np.zeros((1, C, R, S))
        f[0, c0, r0, s0] = 1.0
        got = orc.conv_fwd(x, f, pad=pad)
        P, Q = H + 2 * pad - R + 1, W + 2 * pad - S + 1
        ref = np.zeros((2, 1, P, Q))
        for p in range(P):
            for q in range(Q):
                y, xx = p + r0 - pad, q + s0 - pad
                if 0 <= y < H and 0 <= xx < W:
                    ref[:, 0, p, q] = x[:, c0, y, xx]
        np.testing.assert_array_equal(got, ref)


@pytest.mark.parametrize("shape", SHAPES[:5])
def test_padding_equals_explicit_zero_border(shape):
    x, f, b = _rand(shape, 21)
    st, pad = shape[7], shape[8]
    xp = np.pad(x, ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    np.testing.assert_array_equal(orc.conv_fwd(x, f, b, stride=st, pad=pad), orc.conv_fwd(xp, f, b, stride=st, pad=0))


@pytest.mark.parametrize("st", [2, 3, 4])
def test_stride_subsamples_stride_one(st):
    x, f, b = _rand((2, 3, 14, 15, 4, 3, 5, 1, 1), 31)
    full = orc.conv_fwd(x, f, b, stride=1, pad=1)
    sub = orc.conv_fwd(x, f, b, stride=st, pad=1)
    np.testing.assert_array_equal(sub, full[:, :, ::st, ::st][:, :, :sub.shape[2], :sub.shape[3]])


def test_linearity_batch_independence_channel_permutation():
    shape = (3, 4, 8, 8, 5, 3, 3, 1, 1)
    x, f, b = _rand(shape, 41)
    x2, f2, _ = _rand(shape, 51)
    y = orc.conv_fwd(x, f, pad=1)
    np.testing.assert_allclose(orc.conv_fwd(x + 2 * x2, f, pad=1), y + 2 * orc.conv_fwd(x2, f, pad=1), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.conv_fwd(x, f - 3 * f2, pad=1), y - 3 * orc.conv_fwd(x, f2, pad=1), rtol=1e-12, atol=1e-12)
    # batch items are independent (Section 2)
    for n in range(3):
        np.testing.assert_array_equal(orc.conv_fwd(x[n:n + 1], f, b, pad=1)[0], orc.conv_fwd(x, f, b, pad=1)[n])
    perm = np.array([3, 0, 4, 1, 2])
    np.testing.assert_array_equal(orc.conv_fwd(x, f[perm], b[perm], pad=1), orc.conv_fwd(x, f, b, pad=1)[:, perm])
    # input-channel permutation applied to both operands leaves the result unchanged up to rounding
    cperm = np.array([2, 0, 3, 1])
    np.testing.assert_allclose(orc.conv_fwd(x[:, cperm], f[:, cperm], b, pad=1), orc.conv_fwd(x, f, b, pad=1), rtol=1e-12, atol=1e-13)


def test_relu_properties_and_bias_is_added_before_relu():
    x, f, b = _rand((2, 3, 9, 9, 6, 3, 3, 1, 1), 61)
    lin = orc.conv_fwd(x, f, b, pad=1)
    act = orc.conv_fwd(x, f, b, pad=1, relu=True)
    assert (act >= 0).all() and (lin < 0).any()
    np.testing.assert_array_equal(act, np.maximum(lin, 0.0))
    np.testing.assert_allclose(lin - orc.conv_fwd(x, f, None, pad=1), np.broadcast_to(b[None, :, None, None], lin.shape), rtol=0, atol=1e-12)
    # a large negative bias must zero the output under ReLU (bias after ReLU would leave it negative)
    assert (orc.conv_fwd(x, f, b - 1e6, pad=1, relu=True) == 0).all()


# ---------------------------------------------------------------- library cross-checks
def test_against_scipy_correlate2d():
    from scipy.signal import correlate2d
    x, f, b = _rand((1, 3, 10, 12, 2, 3, 5, 1, 0), 71)
    got = orc.conv_fwd(x, f, b)
    for k in range(2):
        ref = sum(correlate2d(x[0, c], f[k, c], mode="valid") for c in range(3)) + b[k]
        np.testing.assert_allclose(got[0, k], ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("shape", SHAPES)
def test_against_torch_conv2d_fp64(shape):
    import torch
    x, f, b = _rand(shape, 81)
    st, pad = shape[7], shape[8]
    ref = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(f), torch.from_numpy(b), stride=st, padding=pad).numpy()
    np.testing.assert_allclose(orc.conv_fwd(x, f, b, stride=st, pad=pad), ref, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- max-pool
def test_maxpool_hand_case_and_library():
    import torch
    # 5x5 ramp 0..24, 3x3 stride 2 -> windows' maxima are their bottom-right corners
    x = np.arange(25, dtype=np.float64).reshape(1, 1, 5, 5)
    np.testing.assert_array_equal(orc.maxpool_fwd(x)[0, 0], [[12, 14], [22, 24]])
    # negative values: the maximum must not be clamped at zero
    np.testing.assert_array_equal(orc.maxpool_fwd(-x - 1)[0, 0], [[-1, -3], [-11, -13]])
    assert orc.maxpool_fwd(np.zeros((1, 1, 55, 55))).shape == (1, 1, 27, 27)
    assert orc.maxpool_fwd(np.zeros((1, 1, 27, 27))).shape == (1, 1, 13, 13)
    assert orc.maxpool_fwd(np.zeros((1, 1, 13, 13))).shape == (1, 1, 6, 6)
    y = wl.normal(5, (2, 3, 13, 14)).astype(np.float64)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(y), 3, 2).numpy()
    np.testing.assert_array_equal(orc.maxpool_fwd(y), ref)


# ---------------------------------------------------------------- input validation / misc
def test_rejects_windows_that_do_not_fit():
    assert orc.conv_out_dim(2, 3, 1, 0) == 0
    assert orc.conv_out_dim(2, 3, 1, 1) == 2
    assert orc.conv_out_dim(227, 11, 4, 0) == 55
    assert orc.conv_out_dim(10, 3, 2, 0) == 4            # floor((10-3)/2)+1
    with pytest.raises(ValueError):
        orc.conv_fwd(np.zeros((1, 1, 2, 2)), np.zeros((1, 1, 3, 3)))


def test_fp32_inputs_are_widened_exactly():
    x = wl.uniform(9, (1, 2, 5, 5), -1, 1)
    f = wl.normal(10, (3, 2, 3, 3), 0, 0.1)
    assert x.dtype == np.float32
    np.testing.assert_array_equal(orc.conv_fwd(x, f), orc.conv_fwd(x.astype(np.float64), f.astype(np.float64)))


def test_generators_are_deterministic_and_sane():
    a = wl.normal(123, (4000,))
    np.testing.assert_array_equal(a, wl.normal(123, (4000,)))
    assert abs(float(a.mean())) < 0.06 and abs(float(a.std()) - 1.0) < 0.05
    u = wl.uniform(5, (4000,), -1, 1)
    assert u.min() >= -1 and u.max() <= 1 and abs(float(u.mean())) < 0.05
    assert not np.array_equal(wl.normal(123, (10,)), wl.normal(124, (10,)))
    i = wl.integers(3, (1000,))
    assert set(np.unique(i)).issubset(set(range(-8, 9))) and len(np.unique(i)) == 17
    x, w, b = wl.CONFIGS[1].tensors()
    assert x.shape == (1, 3, 32, 32) and w.shape == (16, 3, 3, 3) and b.shape == (16,)
    assert abs(float(w.std()) - 0.1) < 0.02 and abs(float(b.std()) - 0.01) < 0.006
    assert wl.stack_flops(20) == 43065365760
    assert math.isclose(wl.CONFIGS[4].shape.flops, 5980815360)


# ---------------------------------------------------------------- SGEMM oracle (Section 4, Table 1)
def test_sgemm_hand_case():
    # [[1,2],[3,4]] x [[5,6,7],[8,9,10]] worked by hand: row 0 = (1*5+2*8, 1*6+2*9, 1*7+2*10), row 1 likewise
    A = np.array([[1, 2], [3, 4]], dtype=np.float32)
    Bm = np.array([[5, 6, 7], [8, 9, 10]], dtype=np.float32)
    np.testing.assert_array_equal(orc.sgemm(A, Bm), np.array([[21, 24, 27], [47, 54, 61]], dtype=np.float64))


def test_sgemm_closed_forms():
    # ones x ones = K everywhere; identity is neutral on either side; a transposed operand would fail the last check
    M, N, K = 7, 5, 11
    np.testing.assert_array_equal(orc.sgemm(np.ones((M, K)), np.ones((K, N))), np.full((M, N), float(K)))
    X = wl.normal(91, (6, 6))
    np.testing.assert_array_equal(orc.sgemm(np.eye(6), X), X.astype(np.float64))
    np.testing.assert_array_equal(orc.sgemm(X, np.eye(6)), X.astype(np.float64))
    A = np.arange(6, dtype=np.float64).reshape(2, 3)
    Bm = np.arange(12, dtype=np.float64).reshape(3, 4)
    # entry (1, 2): row (3,4,5) . column (2,6,10) = 6 + 24 + 50
    assert orc.sgemm(A, Bm)[1, 2] == 80.0


def test_sgemm_is_the_1x1_convolution():
    # Section 5: a 1x1 convolution of a one-image input is the matrix product filt[M x K] . in[K x N];
    # the two oracle routines are separate loop nests, so each pins the other
    M, N, K = 9, 14, 6
    A = wl.normal(92, (M, K))
    Bm = wl.normal(93, (K, N))
    via_conv = orc.conv_fwd(Bm.reshape(1, K, 1, N), A.reshape(M, K, 1, 1))
    np.testing.assert_allclose(orc.sgemm(A, Bm), via_conv.reshape(M, N), rtol=1e-14, atol=1e-14)


def test_sgemm_against_library_matmul():
    A = wl.normal(94, (33, 17))
    Bm = wl.normal(95, (17, 29))
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    np.testing.assert_allclose(orc.sgemm(A, Bm), ref, rtol=1e-13, atol=1e-13)


# ---- softmax (Section 2 names it among the deployment operations): pins of oracle_softmax_f64
def test_softmax_closed_forms():
    # equal logits -> uniform; [0, ln 3] -> [1/4, 3/4]; [ln 1, ln 2, ln 5] -> [1/8, 2/8, 5/8]
    np.testing.assert_allclose(orc.softmax(np.full((2, 7), 3.25)), np.full((2, 7), 1.0 / 7.0), rtol=1e-15)
    np.testing.assert_allclose(orc.softmax(np.array([[0.0, np.log(3.0)]])), [[0.25, 0.75]], rtol=1e-15)
    np.testing.assert_allclose(orc.softmax(np.log(np.array([[1.0, 2.0, 5.0]]))), [[0.125, 0.25, 0.625]], rtol=1e-15)
    # one column: always 1; rows are independent
    np.testing.assert_array_equal(orc.softmax(np.array([[-4.0], [900.0]])), [[1.0], [1.0]])


def test_softmax_invariants_and_library_cross_check():
    from scipy.special import softmax as sp_softmax
    x = wl.normal(9100, (13, 1000), 0.0, 4.0).astype(np.float64)
    y = orc.softmax(x)
    np.testing.assert_allclose(y.sum(axis=1), 1.0, rtol=1e-14)
    assert (y > 0).all() and (np.argmax(y, axis=1) == np.argmax(x, axis=1)).all()
    np.testing.assert_allclose(orc.softmax(x + 123.5), y, rtol=1e-12)                  # shift invariance
    np.testing.assert_allclose(y[:, 1:] / y[:, :-1], np.exp(x[:, 1:] - x[:, :-1]), rtol=1e-12)   # ratios are exp of differences
    np.testing.assert_allclose(y, sp_softmax(x, axis=1), rtol=1e-13)
    # logits far beyond exp's range in fp64 still give the limit distribution
    np.testing.assert_allclose(orc.softmax(np.array([[1000.0, 1000.0, -1000.0]])), [[0.5, 0.5, 0.0]], atol=1e-300)
    with pytest.raises(ValueError):
        orc.softmax(np.zeros((3,)))
