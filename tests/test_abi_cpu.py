"""CPU-side checks of the C ABI: the library loads, exports what the header declares, and its
host-only helpers and argument validation behave (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

from oracle import conv_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1606_00094_b200.build import build_library
    return ctypes.CDLL(build_library())


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "boda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(boda_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert "boda_conv_fwd" in names and "boda_conv_plan_create" in names and len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/boda.h but not exported"


def test_out_dim_matches_oracle_rule(lib):
    from paper_1606_00094_b200 import binding as B
    for (i, k, s, p) in [(205, 7, 2, 0), (227, 11, 4, 0), (27, 5, 1, 2), (13, 3, 1, 1), (14, 1, 1, 0), (10, 3, 2, 0),
                         (2, 3, 1, 0), (2, 3, 1, 1), (5, 3, 3, 4)]:
        assert B.boda_conv_out_dim(i, k, s, p) == orc.conv_out_dim(i, k, s, p)
    assert B.boda_conv_out_dim(205, 7, 2, 0) == 100     # the paper's worked example, Section 2


def test_argument_validation_needs_no_device():
    from paper_1606_00094_b200 import binding as B
    bad = [(0, 3, 8, 8, 4, 3, 3, 1, 1, 1), (1, 3, 8, 8, 4, 3, 3, 0, 1, 1), (1, 3, 8, 8, 4, 3, 3, 1, -1, 1),
           (1, 3, 2, 2, 4, 3, 3, 1, 0, 1), (1, 3, 8, 8, 0, 3, 3, 1, 1, 1)]
    for s in bad:
        with pytest.raises(B.BodaError) as e:
            B.boda_conv_plan_create(s)
        assert e.value.status == B.BODA_ERR_INVALID_ARG
    with pytest.raises(B.BodaError) as e:
        B.boda_conv_fwd(None, None, None, None, 1, 3, 8, 8, 4, 3, 3, 1, 1, 1, stream=0)
    assert e.value.status == B.BODA_ERR_INVALID_ARG
    with pytest.raises(B.BodaError) as e:
        B.boda_maxpool_fwd(None, None, 1, 1, 5, 5, 3, 2, stream=0)
    assert e.value.status == B.BODA_ERR_INVALID_ARG
    assert B.boda_status_string(0) == "ok" and "timeout" not in B.boda_status_string(1)
    assert B.boda_version() >= 100
    o = B.boda_plan_opts_default()
    assert (o.math, o.tune, o.variant, o.tile_id, o.split_k, o.device, o.s2d) == (0, 0, -1, -1, 0, -1, -1)


def test_run_time_compilation_needs_no_gpu():
    """The run-time specialised DIRECT kernel (Section 4 of the paper) compiles for several shapes on a machine without
    a GPU; the blocking follows the shape."""
    from paper_1606_00094_b200 import binding as B
    try:
        bx, by, smem, image = B.boda_direct_rtc_compile((1, 3, 32, 32, 16, 3, 3, 1, 1, 1), 16)
    except B.BodaError as e:
        if e.status == B.BODA_ERR_UNSUPPORTED:
            pytest.skip("NVRTC is not available on this machine")
        raise
    assert (bx, by) == (32, 8) and smem == 4 * (27 * 16 + 3 * 10 * 35) and image > 1000
    bx, by, smem, image = B.boda_direct_rtc_compile((2, 3, 59, 59, 40, 11, 11, 4, 0, 1), 8)
    assert bx * by >= 32 and smem <= 48 * 1024 and image > 1000
    with pytest.raises(B.BodaError):
        B.boda_direct_rtc_compile((1, 3, 32, 32, 16, 3, 3, 1, 1, 1), 5)            # channels per thread: 4, 8, 16 or 32
    with pytest.raises(B.BodaError):
        B.boda_direct_rtc_compile((1, 256, 13, 13, 64, 3, 3, 1, 1, 1), 16)         # does not fit shared memory
