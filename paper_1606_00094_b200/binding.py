"""Thin ctypes binding of ``libboda.so``: argument marshalling only.

Every function of ``include/boda.h`` is exposed under the same name; tensor arguments may be torch
CUDA tensors (their ``data_ptr()`` is passed) or raw integer addresses.  PyTorch is used for device
memory and streams only; all arithmetic runs in the library's kernels.  There is no CPU fallback:
if the library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

from .build import LIB_PATH

if not os.path.exists(LIB_PATH):
    raise RuntimeError(
        f"{LIB_PATH} is missing: build it with `python -m paper_1606_00094_b200.build` "
        "(there is no CPU fallback)")

_lib = ctypes.CDLL(LIB_PATH)

BODA_OK = 0
BODA_ERR_INVALID_ARG = 1
BODA_ERR_UNSUPPORTED = 2
BODA_ERR_CUDA = 3
BODA_ERR_DEVICE_TIMEOUT = 4
BODA_ERR_NOMEM = 5
BODA_ERR_TOO_LARGE = 6
BODA_VARIANT_AUTO, BODA_VARIANT_DIRECT, BODA_VARIANT_K1CONV, BODA_VARIANT_TCONV = -1, 0, 1, 2
BODA_MATH_AUTO, BODA_MATH_FP32, BODA_MATH_TF32, BODA_MATH_TF32X3, BODA_MATH_F16 = 0, 1, 2, 3, 4
VARIANT_NAMES = {0: "direct", 1: "k1conv", 2: "tconv"}


class boda_conv_shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "C", "H", "W", "K", "R", "S", "stride", "pad", "relu")]


class boda_stack_op(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("conv", boda_conv_shape), ("ksz", ctypes.c_int), ("stride", ctypes.c_int)]


BODA_STACK_CONV, BODA_STACK_MAXPOOL = 0, 1


class boda_plan_opts(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("math", "tune", "variant", "tile_id", "split_k", "device", "s2d")] + \
               [("max_workspace", ctypes.c_size_t)]


_vp = ctypes.c_void_p
_i = ctypes.c_int
_lib.boda_conv_out_dim.argtypes = [_i, _i, _i, _i]
_lib.boda_conv_out_dim.restype = _i
_lib.boda_plan_opts_default.argtypes = [ctypes.POINTER(boda_plan_opts)]
_lib.boda_plan_opts_default.restype = None
_lib.boda_conv_plan_create.argtypes = [ctypes.POINTER(boda_conv_shape), ctypes.POINTER(boda_plan_opts), ctypes.POINTER(_vp)]
_lib.boda_conv_plan_create.restype = _i
_lib.boda_conv_plan_destroy.argtypes = [_vp]
_lib.boda_conv_plan_destroy.restype = _i
_lib.boda_conv_plan_describe.argtypes = [_vp, ctypes.c_char_p, ctypes.c_size_t]
_lib.boda_conv_plan_describe.restype = _i
_lib.boda_conv_plan_workspace_bytes.argtypes = [_vp]
_lib.boda_conv_plan_workspace_bytes.restype = ctypes.c_size_t
_lib.boda_conv_plan_bind_filters.argtypes = [_vp, _vp, _vp]
_lib.boda_conv_plan_bind_filters.restype = _i
_lib.boda_conv_fwd_planned.argtypes = [_vp] * 7
_lib.boda_conv_fwd_planned.restype = _i
_lib.boda_conv_fwd.argtypes = [_vp] * 4 + [_i] * 10 + [_vp]
_lib.boda_conv_fwd.restype = _i
_lib.boda_sgemm.argtypes = [_vp] * 3 + [_i] * 3 + [_vp]
_lib.boda_sgemm.restype = _i
_lib.boda_direct_rtc_compile.argtypes = [ctypes.POINTER(boda_conv_shape), _i, ctypes.POINTER(_i), ctypes.POINTER(_i),
                                         ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
_lib.boda_direct_rtc_compile.restype = _i
_lib.boda_conv_fwd_host.argtypes = [_vp] * 4 + [_i] * 10 + [_vp]
_lib.boda_conv_fwd_host.restype = _i
_lib.boda_conv_fwd_noalloc.argtypes = [_vp] * 4 + [_i] * 10 + [_vp]
_lib.boda_conv_fwd_noalloc.restype = _i
_lib.boda_maxpool_fwd.argtypes = [_vp, _vp] + [_i] * 6 + [_vp]
_lib.boda_maxpool_fwd.restype = _i
_lib.boda_softmax_fwd.argtypes = [_vp, _vp, _i, _i, _vp]
_lib.boda_softmax_fwd.restype = _i
_lib.boda_conv_plan_kernels_per_call.argtypes = [_vp]
_lib.boda_conv_plan_kernels_per_call.restype = _i
_lib.boda_stack_create.argtypes = [ctypes.POINTER(boda_stack_op), _i, ctypes.POINTER(boda_plan_opts), ctypes.POINTER(_vp)]
_lib.boda_stack_create.restype = _i
_lib.boda_stack_create_ex.argtypes = [ctypes.POINTER(boda_stack_op), _i, ctypes.POINTER(boda_plan_opts), ctypes.POINTER(_vp)]
_lib.boda_stack_create_ex.restype = _i
_lib.boda_stack_destroy.argtypes = [_vp]
_lib.boda_stack_destroy.restype = _i
_lib.boda_stack_num_ops.argtypes = [_vp]
_lib.boda_stack_num_ops.restype = _i
_lib.boda_stack_set_filters.argtypes = [_vp, _i, _vp, _vp, _vp]
_lib.boda_stack_set_filters.restype = _i
_lib.boda_stack_out_dims.argtypes = [_vp, _i] + [ctypes.POINTER(_i)] * 4
_lib.boda_stack_out_dims.restype = _i
_lib.boda_stack_copy_layer_output.argtypes = [_vp, _i, _vp, _vp]
_lib.boda_stack_copy_layer_output.restype = _i
_lib.boda_stack_describe.argtypes = [_vp, _i, ctypes.c_char_p, ctypes.c_size_t]
_lib.boda_stack_describe.restype = _i
_lib.boda_stack_kernels_per_fwd.argtypes = [_vp]
_lib.boda_stack_kernels_per_fwd.restype = _i
_lib.boda_stack_fwd.argtypes = [_vp, _vp, _vp, _vp]
_lib.boda_stack_fwd.restype = _i
_lib.boda_stack_fwd_eager.argtypes = [_vp, _vp, _vp, _vp, ctypes.POINTER(_vp)]
_lib.boda_stack_fwd_eager.restype = _i
_lib.boda_stack_run_op.argtypes = [_vp, _i, _vp, _vp, _vp]
_lib.boda_stack_run_op.restype = _i
_lib.boda_stack_fwd_host.argtypes = [_vp, _vp, _vp, _vp]
_lib.boda_stack_fwd_host.restype = _i
_lib.boda_query_status.argtypes = [_vp, ctypes.POINTER(_i)]
_lib.boda_query_status.restype = _i
_lib.boda_clear_caches.argtypes = []
_lib.boda_clear_caches.restype = _i
_lib.boda_status_string.argtypes = [_i]
_lib.boda_status_string.restype = ctypes.c_char_p
_lib.boda_last_error_string.argtypes = []
_lib.boda_last_error_string.restype = ctypes.c_char_p
_lib.boda_kernel_launch_count.argtypes = []
_lib.boda_kernel_launch_count.restype = ctypes.c_ulonglong
_lib.boda_version.argtypes = []
_lib.boda_version.restype = _i


class BodaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.boda_status_string(status).decode()
        detail = _lib.boda_last_error_string().decode() if status == BODA_ERR_CUDA else ""
        super().__init__(f"{where}: {msg}" + (f" [{detail}]" if detail else ""))


def _check(status: int, where: str) -> None:
    if status != BODA_OK:
        raise BodaError(status, where)


def _addr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def boda_version() -> int:
    return int(_lib.boda_version())


def boda_kernel_launch_count() -> int:
    return int(_lib.boda_kernel_launch_count())


def boda_status_string(status: int) -> str:
    return _lib.boda_status_string(status).decode()


def boda_last_error_string() -> str:
    return _lib.boda_last_error_string().decode()


def boda_conv_out_dim(in_dim: int, ksz: int, stride: int, pad: int) -> int:
    return int(_lib.boda_conv_out_dim(in_dim, ksz, stride, pad))


def boda_plan_opts_default() -> boda_plan_opts:
    o = boda_plan_opts()
    _lib.boda_plan_opts_default(ctypes.byref(o))
    return o


def boda_conv_plan_create(shape, opts: Optional[boda_plan_opts] = None) -> int:
    """shape: boda_conv_shape or a 10-tuple (N,C,H,W,K,R,S,stride,pad,relu).  Returns the plan handle."""
    if not isinstance(shape, boda_conv_shape):
        shape = boda_conv_shape(*[int(v) for v in shape])
    handle = _vp()
    _check(_lib.boda_conv_plan_create(ctypes.byref(shape), ctypes.byref(opts) if opts is not None else None,
                                      ctypes.byref(handle)), "boda_conv_plan_create")
    return handle.value


def boda_conv_plan_destroy(plan: int) -> None:
    _check(_lib.boda_conv_plan_destroy(plan), "boda_conv_plan_destroy")


def boda_conv_plan_describe(plan: int) -> str:
    buf = ctypes.create_string_buffer(512)
    _check(_lib.boda_conv_plan_describe(plan, buf, 512), "boda_conv_plan_describe")
    return buf.value.decode()


def boda_conv_plan_workspace_bytes(plan: int) -> int:
    return int(_lib.boda_conv_plan_workspace_bytes(plan))


def boda_conv_plan_bind_filters(plan: int, filt, stream=None) -> None:
    _check(_lib.boda_conv_plan_bind_filters(plan, _addr(filt), _stream(stream)), "boda_conv_plan_bind_filters")


def boda_conv_fwd_planned(plan: int, inp, filt, bias, out, workspace=None, stream=None) -> None:
    _check(_lib.boda_conv_fwd_planned(plan, _addr(inp), _addr(filt), _addr(bias), _addr(out), _addr(workspace),
                                      _stream(stream)), "boda_conv_fwd_planned")


def boda_conv_fwd(inp, filt, bias, out, N, C, H, W, K, R, S, stride, pad, relu, stream=None) -> None:
    _check(_lib.boda_conv_fwd(_addr(inp), _addr(filt), _addr(bias), _addr(out), N, C, H, W, K, R, S, stride, pad,
                              int(bool(relu)), _stream(stream)), "boda_conv_fwd")


def boda_conv_fwd_host(inp, filt, bias, out, N, C, H, W, K, R, S, stride, pad, relu, stream=None) -> None:
    """Same with HOST buffers (torch CPU tensors, preferably pinned, or raw host addresses)."""
    _check(_lib.boda_conv_fwd_host(_addr(inp), _addr(filt), _addr(bias), _addr(out), N, C, H, W, K, R, S, stride, pad,
                                   int(bool(relu)), _stream(stream)), "boda_conv_fwd_host")


BODA_NOALLOC_SCRATCH_BYTES = 32 << 20


def boda_conv_fwd_noalloc(inp, filt, bias, out, N, C, H, W, K, R, S, stride, pad, relu, stream=None) -> None:
    """Forward pass that allocates no device memory: for callers that cannot call cudaMalloc (all device
    memory owned by another allocator, real-time loops, frozen memory budgets).  Scratch lives in a fixed
    array inside the library, shared by all calls: order the calls on one stream.  Raises BodaError with
    BODA_ERR_TOO_LARGE when the shape's scratch exceeds BODA_NOALLOC_SCRATCH_BYTES."""
    _check(_lib.boda_conv_fwd_noalloc(_addr(inp), _addr(filt), _addr(bias), _addr(out), N, C, H, W, K, R, S, stride,
                                      pad, int(bool(relu)), _stream(stream)), "boda_conv_fwd_noalloc")


def boda_direct_rtc_compile(shape, kt):
    """Compiles the run-time specialised DIRECT kernel for `shape` (N,C,H,W,K,R,S,stride,pad,relu) without loading it
    (no GPU needed).  Returns (block_x, block_y, smem_bytes, image_bytes)."""
    s = boda_conv_shape(*shape)
    bx, by = _i(0), _i(0)
    sm, im = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(_lib.boda_direct_rtc_compile(ctypes.byref(s), kt, ctypes.byref(bx), ctypes.byref(by), ctypes.byref(sm),
                                        ctypes.byref(im)), "boda_direct_rtc_compile")
    return bx.value, by.value, sm.value, im.value


def boda_sgemm(A, Bm, C, M, N, K, stream=None) -> None:
    """C[M][N] = A[M][K] @ Bm[K][N], row-major fp32 device tensors."""
    _check(_lib.boda_sgemm(_addr(A), _addr(Bm), _addr(C), M, N, K, _stream(stream)), "boda_sgemm")


def boda_maxpool_fwd(inp, out, N, C, H, W, ksz=3, stride=2, stream=None) -> None:
    _check(_lib.boda_maxpool_fwd(_addr(inp), _addr(out), N, C, H, W, ksz, stride, _stream(stream)), "boda_maxpool_fwd")


def boda_softmax_fwd(inp, out, rows, cols, stream=None) -> None:
    """out[r][:] = softmax(inp[r][:]) for [rows][cols] fp32 device tensors."""
    _check(_lib.boda_softmax_fwd(_addr(inp), _addr(out), rows, cols, _stream(stream)), "boda_softmax_fwd")


def boda_conv_plan_kernels_per_call(plan: int) -> int:
    return int(_lib.boda_conv_plan_kernels_per_call(plan))


def boda_stack_create(ops, opts: Optional[boda_plan_opts] = None) -> int:
    """ops: list of boda_stack_op.  Returns the stack handle."""
    arr = (boda_stack_op * len(ops))(*ops)
    handle = _vp()
    _check(_lib.boda_stack_create(arr, len(ops), ctypes.byref(opts) if opts is not None else None, ctypes.byref(handle)),
           "boda_stack_create")
    return handle.value


def boda_stack_create_ex(ops, per_op_opts) -> int:
    """ops: list of boda_stack_op; per_op_opts: one boda_plan_opts per op.  Returns the stack handle."""
    if len(per_op_opts) != len(ops):
        raise ValueError("one boda_plan_opts per op")
    arr = (boda_stack_op * len(ops))(*ops)
    oarr = (boda_plan_opts * len(ops))(*per_op_opts)
    handle = _vp()
    _check(_lib.boda_stack_create_ex(arr, len(ops), oarr, ctypes.byref(handle)), "boda_stack_create_ex")
    return handle.value


def boda_stack_destroy(stack: int) -> None:
    _check(_lib.boda_stack_destroy(stack), "boda_stack_destroy")


def boda_stack_num_ops(stack: int) -> int:
    return int(_lib.boda_stack_num_ops(stack))


def boda_stack_set_filters(stack: int, op_index: int, filt, bias, stream=None) -> None:
    _check(_lib.boda_stack_set_filters(stack, op_index, _addr(filt), _addr(bias), _stream(stream)), "boda_stack_set_filters")


def boda_stack_out_dims(stack: int, op_index: int):
    v = [_i(0) for _ in range(4)]
    _check(_lib.boda_stack_out_dims(stack, op_index, *[ctypes.byref(x) for x in v]), "boda_stack_out_dims")
    return tuple(x.value for x in v)


def boda_stack_copy_layer_output(stack: int, op_index: int, dst, stream=None) -> None:
    _check(_lib.boda_stack_copy_layer_output(stack, op_index, _addr(dst), _stream(stream)), "boda_stack_copy_layer_output")


def boda_stack_describe(stack: int, op_index: int) -> str:
    buf = ctypes.create_string_buffer(512)
    _check(_lib.boda_stack_describe(stack, op_index, buf, 512), "boda_stack_describe")
    return buf.value.decode()


def boda_stack_kernels_per_fwd(stack: int) -> int:
    return int(_lib.boda_stack_kernels_per_fwd(stack))


def boda_stack_fwd(stack: int, inp, out, stream=None) -> None:
    _check(_lib.boda_stack_fwd(stack, _addr(inp), _addr(out), _stream(stream)), "boda_stack_fwd")


def boda_stack_fwd_eager(stack: int, inp, out, stream=None, events=None) -> None:
    """events: optional flat list of 3 * n_ops torch.cuda.Event objects (already created, timing enabled)."""
    arr = None
    if events is not None:
        handles = []
        for e in events:
            e.record()            # torch creates the underlying cudaEvent lazily: record once to materialise it
            handles.append(e.cuda_event)
        arr = (_vp * len(handles))(*handles)
    _check(_lib.boda_stack_fwd_eager(stack, _addr(inp), _addr(out), _stream(stream), arr), "boda_stack_fwd_eager")


def boda_stack_run_op(stack: int, op_index: int, inp=None, out=None, stream=None) -> None:
    _check(_lib.boda_stack_run_op(stack, op_index, _addr(inp), _addr(out), _stream(stream)), "boda_stack_run_op")


def boda_stack_fwd_host(stack: int, inp_host, out_host, stream=None) -> None:
    _check(_lib.boda_stack_fwd_host(stack, _addr(inp_host), _addr(out_host), _stream(stream)), "boda_stack_fwd_host")


def boda_query_status(stream=None) -> int:
    st = _i(0)
    _check(_lib.boda_query_status(_stream(stream), ctypes.byref(st)), "boda_query_status")
    return st.value


def boda_clear_caches() -> None:
    _check(_lib.boda_clear_caches(), "boda_clear_caches")


# ---------------------------------------------------------------------------------------------------
# Conveniences on top of the ABI (allocation through torch; no arithmetic).

class ConvPlan:
    """Owns a plan handle and its workspace; ``plan(x, w, b)`` runs the layer into a new tensor."""

    def __init__(self, shape, math=BODA_MATH_AUTO, variant=BODA_VARIANT_AUTO, tile_id=-1, split_k=0, tune=0, s2d=-1,
                 max_workspace=0):
        import torch
        self.shape = tuple(int(v) for v in shape)
        o = boda_plan_opts_default()
        o.math, o.variant, o.tile_id, o.split_k, o.tune, o.s2d = math, variant, tile_id, split_k, tune, s2d
        o.max_workspace = max_workspace
        self.handle = boda_conv_plan_create(self.shape, o)
        nbytes = boda_conv_plan_workspace_bytes(self.handle)
        self.workspace = torch.empty(max(nbytes, 1), dtype=torch.uint8, device="cuda") if nbytes else None
        N, C, H, W, K, R, S, stride, pad, _ = self.shape
        self.out_shape = (N, K, boda_conv_out_dim(H, R, stride, pad), boda_conv_out_dim(W, S, stride, pad))

    def describe(self) -> str:
        return boda_conv_plan_describe(self.handle)

    def bind_filters(self, filt, stream=None) -> None:
        boda_conv_plan_bind_filters(self.handle, filt, stream)

    def __call__(self, x, filt, bias=None, out=None, stream=None):
        import torch
        if out is None:
            out = torch.empty(self.out_shape, dtype=torch.float32, device=x.device)
        boda_conv_fwd_planned(self.handle, x, filt, bias, out, self.workspace, stream)
        return out

    def close(self) -> None:
        if self.handle:
            boda_conv_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def conv_fwd(x, filt, bias=None, stride=1, pad=0, relu=True, stream=None):
    """One-call forward on CUDA tensors via ``boda_conv_fwd`` (plan cached inside the library)."""
    import torch
    N, C, H, W = x.shape
    K, _, R, S = filt.shape
    out = torch.empty((N, K, boda_conv_out_dim(H, R, stride, pad), boda_conv_out_dim(W, S, stride, pad)),
                      dtype=torch.float32, device=x.device)
    boda_conv_fwd(x, filt, bias, out, N, C, H, W, K, R, S, stride, pad, relu, stream)
    return out


def maxpool_fwd(x, ksz=3, stride=2, stream=None):
    import torch
    N, C, H, W = x.shape
    out = torch.empty((N, C, boda_conv_out_dim(H, ksz, stride, 0), boda_conv_out_dim(W, ksz, stride, 0)),
                      dtype=torch.float32, device=x.device)
    boda_maxpool_fwd(x, out, N, C, H, W, ksz, stride, stream)
    return out
