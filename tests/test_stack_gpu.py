"""The AlexNet-shaped conv stack end to end on the GPU against the fp64 oracle chain."""
import numpy as np
import pytest

from oracle import conv_oracle as orc
from paper_1606_00094_b200 import workloads as wl
from helpers import FP32_TOL, TF32_TOL

pytestmark = pytest.mark.gpu


def _oracle_chain(x, params, ops):
    """fp64 end to end: layer i feeds layer i+1 without ever being rounded to fp32."""
    outs = []
    a = x.astype(np.float64)
    it = iter(params)
    for op in ops:
        if op.kind == "conv":
            w, b = next(it)
            s = op.shape
            a = orc.conv_fwd(a, w, b, stride=s.stride, pad=s.pad, relu=True)
        else:
            a = orc.maxpool_fwd(a, op.ksz, op.stride)
        outs.append(a)
    return outs


# (20, auto, tuned) is the launch configuration bench.py times; math 3 is the error-compensated TF32 mode, which
# must hold the FP32 bar through the whole chain (its layers hand over in NCHW)
@pytest.mark.parametrize("batch,math,tol,tune", [(2, 0, TF32_TOL, 0), (1, 1, FP32_TOL, 0), (20, 0, TF32_TOL, 0),
                                                 (20, 0, TF32_TOL, 1), (2, 3, FP32_TOL, 0)])
def test_stack_every_layer_matches_fp64_chain(batch, math, tol, tune):
    import torch
    from paper_1606_00094_b200 import binding as B
    from paper_1606_00094_b200.stack import ConvStack
    ops = wl.alexnet_stack(batch)
    x, params = wl.stack_tensors(batch)
    ref = _oracle_chain(x, params, ops)
    stack = ConvStack(ops, params, math=math, tune=tune)
    try:
        dx = torch.from_numpy(x).cuda()
        out_graph = stack.forward(dx).clone()            # first call: eager pass + graph capture + launch
        out_graph2 = stack.forward(dx).clone()           # pure graph replay
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0
        assert torch.equal(out_graph, out_graph2)
        descs = stack.describe()
        for i, r in enumerate(ref):
            got = stack.layer_output(i)
            if got is None:                              # pooled inside the epilogue: checked through the pool's output
                assert "maxpool" in descs[i] and "fused" in descs[i + 1]
                continue
            got = got.cpu().numpy()
            assert got.shape == r.shape
            err = orc.rel_l2(got, r)
            assert err <= tol, f"op {i} ({descs[i]}): rel-L2 {err:.3e} > {tol:.0e}"
        # host-buffer entry point: from batch 4 on it runs the batch in slices through plans made for the sub-batch
        # (copies overlap kernels), so it is held to the oracle like the device path, and to itself bit for bit;
        # smaller batches take the very same graph
        hx = torch.from_numpy(x).pin_memory()
        ho = torch.empty(stack.out_shape, dtype=torch.float32).pin_memory()
        ho2 = torch.empty(stack.out_shape, dtype=torch.float32).pin_memory()
        stack.forward_host(hx, ho)
        stack.forward_host(hx, ho2)
        assert B.boda_query_status() == 0
        assert torch.equal(ho, ho2)
        if batch < 4:
            assert torch.equal(ho, out_graph.cpu())
        else:
            err = orc.rel_l2(ho.numpy(), ref[-1])
            assert err <= tol, f"host path: rel-L2 {err:.3e} > {tol:.0e}"
        eager = stack.forward_eager(dx).clone()
        torch.cuda.synchronize()
        assert torch.equal(eager, out_graph)
        if math == 0:
            assert any("tconv" in d for d in descs)
        elif math == 3:
            assert any("tf32x3" in d for d in descs)
        else:
            assert all("direct" in d or "maxpool" in d for d in descs)
        assert stack.kernels_per_forward() >= len(ops) - sum("fused" in d for d in descs)
    finally:
        stack.close()


@pytest.mark.parametrize("batch,tune,fuse", [(2, 0, True), (20, 1, True), (20, 0, False)])
def test_stack_layers_in_isolation(batch, tune, fuse, monkeypatch):
    """Every GPU layer against the oracle layer applied to the GPU's OWN input of that layer (so an error cannot be
    blamed on, or hidden by, the layers before it): pooling is compare-and-index work and must be bit-exact in
    every layout the chain uses; convolutions meet the TF32 bar.  (20, tuned) is what bench.py times."""
    import torch
    from paper_1606_00094_b200 import binding as B
    from paper_1606_00094_b200.stack import ConvStack
    if not fuse:
        monkeypatch.setenv("BODA_STACK_NO_POOL_FUSION", "1")     # every pool as a kernel of its own
    ops = wl.alexnet_stack(batch)
    x, params = wl.stack_tensors(batch)
    stack = ConvStack(ops, params, tune=tune)
    try:
        stack.forward(torch.from_numpy(x).cuda())
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0
        descs = stack.describe()
        prev = x
        it = iter(params)
        pending = None                                   # oracle output of a convolution the GPU did not materialise
        for i, op in enumerate(ops):
            got = stack.layer_output(i)
            got = None if got is None else got.cpu().numpy()
            if op.kind == "conv":
                w, b = next(it)
                s = op.shape
                ref = orc.conv_fwd(prev, w, b, stride=s.stride, pad=s.pad, relu=True)
                if got is None:                          # the pool runs in this layer's epilogue: judged on the pooled tensor
                    pending = ref
                    continue
                err = orc.rel_l2(got, ref)
                assert err <= TF32_TOL, f"op {i} ({descs[i]}): rel-L2 {err:.3e}"
            elif pending is not None:
                ref = orc.maxpool_fwd(pending, op.ksz, op.stride)
                err = orc.rel_l2(got, ref)
                assert err <= TF32_TOL, f"op {i - 1}+{i} ({descs[i - 1]}): rel-L2 {err:.3e}"
                pending = None
            else:
                ref = orc.maxpool_fwd(prev, op.ksz, op.stride)
                np.testing.assert_array_equal(got.astype(np.float64), ref, err_msg=f"op {i} ({descs[i]})")
            prev = got
    finally:
        stack.close()


def test_forward_host_is_ordered_behind_earlier_work_on_the_stream():
    """The host-buffer entry point copies its input on a second stream; that stream must wait for what the caller
    queued on `stream` before the call.  Here the pinned input buffer is itself filled by a device-to-host copy queued
    behind a long-running kernel: if the slices were read early, the chain would see the stale zeros."""
    import torch
    from paper_1606_00094_b200 import binding as B
    from paper_1606_00094_b200.stack import ConvStack
    batch = 4                                           # sliced path (even batch >= 4)
    ops = wl.alexnet_stack(batch)
    x, params = wl.stack_tensors(batch)
    stack = ConvStack(ops, params)
    try:
        dx = torch.from_numpy(x).cuda()
        want = torch.empty(stack.out_shape, dtype=torch.float32).pin_memory()
        hx_ready = torch.from_numpy(x).pin_memory()
        stack.forward_host(hx_ready, want)              # reference result (also creates the sub-batch stack)
        hx = torch.zeros(x.shape, dtype=torch.float32).pin_memory()
        got = torch.empty(stack.out_shape, dtype=torch.float32).pin_memory()
        torch.cuda.synchronize()
        torch.cuda._sleep(200_000_000)                  # about 0.1 s of GPU time on the current stream
        hx.copy_(dx, non_blocking=True)                 # fills the pinned input once the sleep has ended
        stack.forward_host(hx, got)
        assert B.boda_query_status() == 0
        assert torch.equal(hx, hx_ready)
        assert torch.equal(got, want), "the input slices were copied before the stream's earlier work had finished"
    finally:
        stack.close()


def test_stack_rejects_shapes_that_do_not_chain():
    from paper_1606_00094_b200 import binding as B
    a = B.boda_stack_op()
    a.kind = B.BODA_STACK_CONV
    a.conv = B.boda_conv_shape(1, 3, 16, 16, 8, 3, 3, 1, 1, 1)
    b = B.boda_stack_op()
    b.kind = B.BODA_STACK_CONV
    b.conv = B.boda_conv_shape(1, 4, 16, 16, 8, 3, 3, 1, 1, 1)      # expects 4 channels, gets 8
    with pytest.raises(B.BodaError) as e:
        B.boda_stack_create([a, b])
    assert e.value.status == B.BODA_ERR_INVALID_ARG
