"""Shared helpers of the GPU parity tests: run a layer through the C ABI and compare with the oracle."""
import numpy as np

from oracle import conv_oracle as orc

GUARD = 1024  # floats of NaN guard band on each side of the output buffer
FP32_TOL = 1e-5   # relative L2 bar of the FP32 CUDA-core path
TF32_TOL = 5e-3   # relative L2 bar of the TF32 tensor-core path


def run_planned(shape, x, w, b, *, variant=-1, math=0, tile_id=-1, split_k=0, bind=False, tune=0, s2d=-1):
    """shape = (N,C,H,W,K,R,S,stride,pad,relu); x,w,b numpy fp32.  Returns (out numpy, description)."""
    import torch
    from paper_1606_00094_b200 import binding as B
    plan = B.ConvPlan(shape, math=math, variant=variant, tile_id=tile_id, split_k=split_k, tune=tune, s2d=s2d)
    try:
        dx = torch.from_numpy(x).cuda()
        dw = torch.from_numpy(w).cuda()
        db = torch.from_numpy(b).cuda() if b is not None else None
        n_out = int(np.prod(plan.out_shape))
        buf = torch.full((n_out + 2 * GUARD,), float("nan"), dtype=torch.float32, device="cuda")
        out = buf[GUARD:GUARD + n_out].view(plan.out_shape)
        if bind:
            plan.bind_filters(dw)
        plan(dx, dw, db, out=out)
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0, "device status word set"
        host = buf.cpu().numpy()
        assert np.isnan(host[:GUARD]).all() and np.isnan(host[GUARD + n_out:]).all(), "guard band overwritten"
        res = host[GUARD:GUARD + n_out].reshape(plan.out_shape).copy()
        assert not np.isnan(res).any(), "output not fully written"
        return res, plan.describe()
    finally:
        plan.close()


def oracle_out(shape, x, w, b):
    N, C, H, W, K, R, S, stride, pad, relu = shape
    return orc.conv_fwd(x, w, b, stride=stride, pad=pad, relu=bool(relu))


def assert_parity(got, ref, tol, what=""):
    err = orc.rel_l2(got, ref)
    assert err <= tol, f"{what}: rel-L2 {err:.3e} > {tol:.1e} (max abs {np.abs(got - ref).max():.3e})"
    return err
