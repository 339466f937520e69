"""Element-exact parity of chained layers: the staged hand-off between tensor-core kernels and the pooling kernels
that read and write the staged layout - the configuration the benchmark's step runs.

Operands are drawn from {-1, 0, 1}.  Then every product and partial sum is an integer, the first layer's outputs stay
below 2048 (exactly representable in TF32, so the rounding the producing epilogue applies to a staged activation
changes nothing) and later sums stay below 2^24 (exact in fp32): every layer of the GPU chain must EQUAL the fp64
oracle chain, element by element - a misplaced or dropped element cannot hide behind a tolerance.
"""
import numpy as np
import pytest

from oracle import conv_oracle as orc
from paper_1606_00094_b200 import workloads as wl
from paper_1606_00094_b200.workloads import ConvShape, StackOp

pytestmark = pytest.mark.gpu

# tile ids of the tensor-core variants: 0..4 im2col tiles 128x64/96/128/192/256, 5.. halo tiles
IM2COL_64, IM2COL_128, IM2COL_192 = 0, 2, 3
HALO_128x64, HALO_128x128, HALO_256x96, HALO_256x128, HALO_512x64, HALO_512x96 = 5, 6, 9, 10, 13, 14


def _ternary(seed, shape):
    return wl.integers(seed, shape, -1, 1)


def _oracle_chain(x, params, ops):
    outs = []
    a = x.astype(np.float64)
    it = iter(params)
    for op in ops:
        if op.kind == "conv":
            w, b = next(it)
            s = op.shape
            a = orc.conv_fwd(a, w, b, stride=s.stride, pad=s.pad, relu=bool(s.relu))
        else:
            a = orc.maxpool_fwd(a, op.ksz, op.stride)
        outs.append(a)
    return outs


def _run_chain_exact(ops, per_op, seed, expect):
    import torch
    from paper_1606_00094_b200 import binding as B
    from paper_1606_00094_b200.stack import ConvStack
    first = ops[0].shape
    x = _ternary(seed, (first.N, first.C, first.H, first.W))
    params = []
    for i, op in enumerate(ops):
        if op.kind == "conv":
            s = op.shape
            params.append((_ternary(seed + 10 * i + 1, (s.K, s.C, s.R, s.S)), _ternary(seed + 10 * i + 2, (s.K,))))
    ref = _oracle_chain(x, params, ops)
    for r in ref[:-1]:
        assert np.abs(r).max() <= 2048, "test design: a staged activation must be exact in TF32"
    assert np.abs(ref[-1]).max() < 2 ** 24
    stack = ConvStack(ops, params, per_op=per_op)
    try:
        descs = stack.describe()
        for i, want in expect.items():
            for frag in want:
                assert frag in descs[i], f"op {i}: wanted '{frag}' in '{descs[i]}'"
        out = stack.forward(torch.from_numpy(x).cuda()).clone()
        out2 = stack.forward(torch.from_numpy(x).cuda()).clone()
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0
        assert torch.equal(out, out2)
        for i, r in enumerate(ref):
            got = stack.layer_output(i)
            if got is None:                 # a convolution whose pool runs in its epilogue: only the pooled tensor exists
                assert "fused" in descs[i + 1]
                continue
            np.testing.assert_array_equal(got.cpu().numpy().astype(np.float64), r, err_msg=f"op {i}: {descs[i]}")
    finally:
        stack.close()


# conv -> conv hand-off, both 3x3 pad 1 on 13x13 (tiles straddle rows and images): C = 40 is not a multiple of 32
# (padded channels of the staged input), K = 72 gives a staged activation whose 96 channels exceed the producer's 64
# (im2col tile of 64 columns: the second column tile is ragged)
CONV_CONV = [
    # (tile, split) of the producer, (tile, split) of the consumer
    ((IM2COL_64, 1), (IM2COL_64, 1)),
    ((IM2COL_128, 2), (IM2COL_64, 2)),
    ((IM2COL_192, 1), (HALO_128x64, 1)),
    ((HALO_128x128, 1), (IM2COL_128, 1)),
    ((HALO_256x96, 1), (HALO_256x128, 1)),
    ((HALO_128x64, 2), (HALO_128x128, 2)),
    ((HALO_512x96, 1), (HALO_512x64, 1)),
]


@pytest.mark.parametrize("prod,cons", CONV_CONV)
def test_conv_to_conv_staged_handoff_is_exact(prod, cons):
    ops = [StackOp("conv", ConvShape(3, 40, 13, 13, 72, 3, 3, 1, 1, True)),
           StackOp("conv", ConvShape(3, 72, 13, 13, 48, 3, 3, 1, 1, False))]
    per_op = [{"variant": 2, "tile_id": prod[0], "split_k": prod[1]}, {"variant": 2, "tile_id": cons[0], "split_k": cons[1]}]
    _run_chain_exact(ops, per_op, 900, {0: ["out=staged", f"id {prod[0]}"], 1: ["in=staged", f"id {cons[0]}"]})


# conv -> pool -> conv -> pool: the pooling kernels on the staged layout (staged -> staged, staged -> NCHW); the first
# convolution has no ReLU so that the first pool sees negative values
CONV_POOL = [
    ((IM2COL_64, 1), (IM2COL_64, 1)),
    ((IM2COL_128, 2), (HALO_128x64, 1)),
    ((HALO_256x96, 1), (IM2COL_128, 2)),
    ((HALO_128x128, 2), (HALO_256x128, 1)),
]


@pytest.mark.parametrize("prod,cons", CONV_POOL)
def test_conv_pool_conv_pool_staged_is_exact(prod, cons, monkeypatch):
    monkeypatch.setenv("BODA_STACK_NO_POOL_FUSION", "1")          # the pooling kernels themselves are under test here
    ops = [StackOp("conv", ConvShape(2, 24, 19, 19, 40, 3, 3, 1, 1, False)),
           StackOp("pool"),                                                            # 19 -> 9
           StackOp("conv", ConvShape(2, 40, 9, 9, 72, 3, 3, 1, 1, True)),
           StackOp("pool")]                                                            # 9 -> 4, NCHW out
    per_op = [{"variant": 2, "tile_id": prod[0], "split_k": prod[1]}, {},
              {"variant": 2, "tile_id": cons[0], "split_k": cons[1]}, {}]
    _run_chain_exact(ops, per_op, 1200, {0: ["out=staged"], 1: ["in=staged", "out=staged"], 2: ["in=staged", "out=staged"],
                                         3: ["in=staged", "out=nchw"]})


# The same chain with the pools run inside the convolutions' epilogues (halo tiles of 256 or 512 positions, no split):
# tiles then follow whole output rows of one image, and the pooled tensor is written in the consumer's staged layout
# (first pool) or as NCHW (last pool).  19 x 19 -> 9 x 9 pooled: tiles of 256 positions hold 4 pooled rows (ragged
# last tile), of 512 positions all 9.
FUSED = [
    ((HALO_256x96, 1), (HALO_256x128, 1)),
    ((HALO_512x96, 1), (HALO_512x64, 1)),
    ((HALO_256x128, 1), (IM2COL_128, 1)),          # the consumer's pool stays a kernel of its own (im2col tile)
]


@pytest.mark.parametrize("prod,cons", FUSED)
def test_fused_pool_epilogue_is_exact(prod, cons):
    ops = [StackOp("conv", ConvShape(2, 24, 19, 19, 40, 3, 3, 1, 1, True)),
           StackOp("pool"),
           StackOp("conv", ConvShape(2, 40, 9, 9, 72, 3, 3, 1, 1, True)),
           StackOp("pool")]
    per_op = [{"variant": 2, "tile_id": prod[0], "split_k": prod[1]}, {},
              {"variant": 2, "tile_id": cons[0], "split_k": cons[1]}, {}]
    halo_cons = cons[0] >= 5
    _run_chain_exact(ops, per_op, 1300, {0: ["+maxpool3x3s2"], 1: ["fused"], 2: ["in=staged"] + (["+maxpool3x3s2"] if halo_cons else []),
                                         3: ["fused"] if halo_cons else ["in=staged", "out=nchw"]})


# a first layer on 3 channels with a strided window through its space-to-depth view (NCHW in, halo tile, staged
# out), pooled, then a 5x5 layer: the shape of the AlexNet-shaped stack's first three ops, small
FIRST_512x64, FIRST_512x96 = 23, 24       # the first-layer kernel: no staged input at all


@pytest.mark.parametrize("first,second", [((HALO_512x96, 1), (IM2COL_128, 1)), ((HALO_256x96, 1), (HALO_128x128, 1)),
                                          ((FIRST_512x96, 1), (IM2COL_128, 1)), ((FIRST_512x64, 1), (HALO_128x128, 1))])
def test_space_to_depth_first_layer_pool_conv_is_exact(first, second):
    ops = [StackOp("conv", ConvShape(2, 3, 67, 67, 80, 11, 11, 4, 0, True)),           # -> 15 x 15
           StackOp("pool"),                                                            # -> 7 x 7
           StackOp("conv", ConvShape(2, 80, 7, 7, 48, 5, 5, 1, 2, True))]
    per_op = [{"variant": 2, "tile_id": first[0], "split_k": first[1], "s2d": 1}, {},
              {"variant": 2, "tile_id": second[0], "split_k": second[1]}]
    _run_chain_exact(ops, per_op, 1500, {0: ["s2d", "in=nchw", "out=staged", "+maxpool3x3s2"], 1: ["fused"], 2: ["in=staged"]})


def test_default_plans_chain_is_exact():
    """No forced tiles: whatever the rules pick for an AlexNet-like (small) chain must hand over exactly."""
    ops = [StackOp("conv", ConvShape(2, 3, 67, 67, 64, 11, 11, 4, 0, True)),
           StackOp("pool"),
           StackOp("conv", ConvShape(2, 64, 7, 7, 96, 5, 5, 1, 2, True)),
           StackOp("conv", ConvShape(2, 96, 7, 7, 64, 3, 3, 1, 1, True)),
           StackOp("pool")]
    # three convolutions: the second and third have sparse filters so that every staged activation stays exact in TF32
    import torch  # noqa: F401  (the chain runs on the GPU)
    from paper_1606_00094_b200 import binding as B
    from paper_1606_00094_b200.stack import ConvStack
    x = _ternary(1700, (2, 3, 67, 67))
    w1, b1 = _ternary(1701, (64, 3, 11, 11)), _ternary(1702, (64,))
    w2 = _ternary(1703, (96, 64, 5, 5)) * (wl.uniform01(1704, 96 * 64 * 25).reshape(96, 64, 5, 5) < 0.05)
    w2 = w2.astype(np.float32)
    b2 = _ternary(1705, (96,))
    w3 = _ternary(1706, (64, 96, 3, 3)) * (wl.uniform01(1708, 64 * 96 * 9).reshape(64, 96, 3, 3) < 0.05)
    w3 = w3.astype(np.float32)
    b3 = _ternary(1707, (64,))
    params = [(w1, b1), (w2, b2), (w3, b3)]
    ref = _oracle_chain(x, params, ops)
    for r in ref[:-1]:
        assert np.abs(r).max() <= 2048
    stack = ConvStack(ops, params)
    try:
        import torch
        out = stack.forward(torch.from_numpy(x).cuda())
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0
        descs = stack.describe()
        for i, r in enumerate(ref):
            got = stack.layer_output(i).cpu().numpy().astype(np.float64)
            np.testing.assert_array_equal(got, r, err_msg=f"op {i}: {descs[i]}")
        assert out.shape == ref[-1].shape
    finally:
        stack.close()
