"""GPU softmax against the fp64 oracle."""
import numpy as np
import pytest

from oracle import conv_oracle as orc
from paper_1606_00094_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols,scale", [(20, 1000, 4.0), (1, 1, 1.0), (3, 7, 30.0), (5, 256, 1.0), (2, 11264, 3.0),
                                             (2, 20000, 3.0), (64, 33, 80.0)])
def test_softmax_matches_oracle(rows, cols, scale):
    import torch
    from paper_1606_00094_b200 import binding as B
    x = wl.normal(9200 + cols, (rows, cols), 0.0, scale)
    ref = orc.softmax(x)
    dx = torch.from_numpy(x).cuda()
    out = torch.full((rows, cols), float("nan"), dtype=torch.float32, device="cuda")
    B.boda_softmax_fwd(dx, out, rows, cols)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    # fp32 exp and an fp32 sum of up to 20000 terms: a few units in the seventh digit
    assert orc.rel_l2(got, ref) <= 2e-6
    np.testing.assert_allclose(got.sum(axis=1), 1.0, rtol=2e-6)
    assert (np.argmax(got, axis=1) == np.argmax(ref, axis=1)).all()
    B.boda_softmax_fwd(dx, dx, rows, cols)                     # in place
    torch.cuda.synchronize()
    np.testing.assert_array_equal(dx.cpu().numpy(), out.cpu().numpy())


def test_softmax_extreme_logits_and_bad_arguments():
    import torch
    from paper_1606_00094_b200 import binding as B
    x = torch.tensor([[1000.0, 1000.0, -1000.0], [-3e38, 0.0, -3e38]], device="cuda")
    out = torch.empty_like(x)
    B.boda_softmax_fwd(x, out, 2, 3)
    torch.cuda.synchronize()
    np.testing.assert_allclose(out.cpu().numpy(), [[0.5, 0.5, 0.0], [0.0, 1.0, 0.0]], atol=1e-7)
    with pytest.raises(B.BodaError):
        B.boda_softmax_fwd(x, out, 0, 3)
