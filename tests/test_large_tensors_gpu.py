"""Tensors of a gigabyte and more: element offsets near 2^30 and byte offsets past 2^31 and 2^32.

The oracle cannot run such a layer whole in seconds, so inputs are a closed-form function of the flat element index
(small integers: every product and partial sum is exact in TF32 and fp32), generated on the device in pieces, and
the oracle's definition is evaluated output by output on a sample that includes the first and last elements and the
neighbourhood of every power-of-two byte offset.  Bit-exact equality is required.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _value(idx, mul, mod):
    """integer-valued tensor entry for flat index idx (numpy int64 array or scalar): in [-(mod//2), mod//2]"""
    return ((idx * mul + 7) % mod) - (mod // 2)


def _fill(t, mul, mod):
    import torch
    flat = t.view(-1)
    step = 1 << 26
    for s in range(0, flat.numel(), step):
        e = min(flat.numel(), s + step)
        i = torch.arange(s, e, dtype=torch.int64, device=t.device)
        flat[s:e] = (((i * mul + 7) % mod) - (mod // 2)).to(torch.float32)


def _oracle_point(shape, n, k, p, q):
    """the definition of Section 2 for one output element, inputs recomputed from their closed form"""
    N, C, H, W, K, R, S, stride, pad, relu = shape
    acc = float(_value(np.int64(k), 5, 9))                                         # bias[k]
    for c in range(C):
        for r in range(R):
            y = p * stride + r - pad
            if y < 0 or y >= H:
                continue
            for s in range(S):
                x = q * stride + s - pad
                if x < 0 or x >= W:
                    continue
                xi = ((np.int64(n) * C + c) * H + y) * W + x
                wi = ((np.int64(k) * C + c) * R + r) * S + s
                acc += float(_value(xi, 2654435761, 17)) * float(_value(wi, 40503, 5))
    return max(acc, 0.0) if relu else acc


def _sample_points(shape, count, rng):
    N, C, H, W, K, R, S, stride, pad, relu = shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    total = N * K * P * Q
    flats = {0, 1, total - 1, total - 2}
    for bits in (27, 28, 29, 30, 31):                          # element offsets whose byte offsets cross 2^29 .. 2^33
        for d in (-1, 0, 1):
            f = (1 << bits) + d
            if 0 <= f < total:
                flats.add(f)
    flats.update(int(v) for v in rng.integers(0, total, size=count))
    pts = []
    for f in sorted(flats):
        q = f % Q; t = f // Q
        p = t % P; t //= P
        k = t % K; n = t // K
        pts.append((f, n, k, p, q))
    return pts, (N, K, P, Q)


CASES = [
    # shape, variant (-1 auto), tile, math
    ((4096, 64, 64, 64, 64, 1, 1, 1, 0, 1), 1, -1, 0),        # 1.07 G elements in and out (4.3 GB each): the NCHW 1x1 kernel
    ((4096, 64, 64, 64, 64, 1, 1, 1, 0, 1), 1, 2, 0),         # the same through the staged path (4.3 GB workspace)
    ((4096, 64, 64, 64, 64, 1, 1, 1, 0, 1), 1, 19, 0),        # the gather kernel
    ((2048, 32, 128, 128, 32, 3, 3, 1, 1, 1), 2, -1, 0),      # 3x3 with padding, 1.07 G elements in and out
    ((1024, 3, 256, 256, 16, 3, 3, 1, 1, 1), 0, -1, 1),       # FP32 kernel (run-time compiled where NVRTC is there): 1.07 G outputs
]


@pytest.mark.parametrize("shape,variant,tile,math", CASES)
def test_offsets_past_32_bits(shape, variant, tile, math):
    import torch
    from paper_1606_00094_b200 import binding as B
    N, C, H, W, K, R, S, stride, pad, relu = shape
    free, _ = torch.cuda.mem_get_info()
    if free < 24 * (1 << 30):
        pytest.skip("needs 24 GB of free device memory")
    x = torch.empty((N, C, H, W), dtype=torch.float32, device="cuda")
    w = torch.empty((K, C, R, S), dtype=torch.float32, device="cuda")
    b = torch.empty((K,), dtype=torch.float32, device="cuda")
    _fill(x, 2654435761, 17)
    _fill(w, 40503, 5)
    _fill(b, 5, 9)
    plan = B.ConvPlan(shape, variant=variant, tile_id=tile, math=math)
    try:
        out = torch.full(plan.out_shape, float("nan"), dtype=torch.float32, device="cuda")
        plan(x, w, b, out=out)
        torch.cuda.synchronize()
        assert B.boda_query_status() == 0
        desc = plan.describe()
        pts, dims = _sample_points(shape, 150, np.random.default_rng(1606))
        assert tuple(out.shape) == dims
        flat = out.view(-1)
        idx = torch.tensor([f for f, *_ in pts], dtype=torch.int64, device="cuda")
        got = flat[idx].cpu().numpy().astype(np.float64)
        ref = np.array([_oracle_point(shape, n, k, p, q) for _, n, k, p, q in pts])
        np.testing.assert_array_equal(got, ref, err_msg=desc)
        assert not torch.isnan(flat[:: 4099]).any(), "output not fully written"      # a coarse sweep over the whole tensor
    finally:
        plan.close()
        del x, w, b
        torch.cuda.empty_cache()
