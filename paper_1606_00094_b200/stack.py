"""Python face of ``boda_stack``: a chain of convolution and pooling layers run as one CUDA graph.

Marshalling only: the chain, its plans, activations, workspace and graph live in the library
(``csrc/stack.cu``); this class keeps the filter tensors alive and hands out torch views.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B
from .workloads import StackOp


class ConvStack:
    def __init__(self, ops: Sequence[StackOp], params: Sequence[Tuple], math: int = B.BODA_MATH_AUTO,
                 tune: int = 0, device: str = "cuda", per_op: Optional[Sequence[dict]] = None):
        """ops: conv / pool descriptors; params: per conv layer (filters, bias) as numpy fp32 arrays;
        per_op: optional plan options per op (dicts with keys of boda_plan_opts, e.g. tile_id, split_k, s2d)."""
        self.ops = list(ops)
        c_ops = []
        for op in self.ops:
            o = B.boda_stack_op()
            if op.kind == "conv":
                o.kind = B.BODA_STACK_CONV
                o.conv = B.boda_conv_shape(*op.shape.as_tuple())
            else:
                o.kind = B.BODA_STACK_MAXPOOL
                o.ksz, o.stride = op.ksz, op.stride
            c_ops.append(o)
        if per_op is None:
            opts = B.boda_plan_opts_default()
            opts.math, opts.tune = math, tune
            self.handle = B.boda_stack_create(c_ops, opts)
        else:
            all_opts = []
            for d in per_op:
                o = B.boda_plan_opts_default()
                o.math, o.tune = math, tune
                for k, v in (d or {}).items():
                    setattr(o, k, v)
                all_opts.append(o)
            self.handle = B.boda_stack_create_ex(c_ops, all_opts)
        self.filters: List[Optional[torch.Tensor]] = []
        self.biases: List[Optional[torch.Tensor]] = []
        it = iter(params)
        for i, op in enumerate(self.ops):
            if op.kind == "conv":
                w, b = next(it)
                fw = torch.from_numpy(w).to(device)
                fb = torch.from_numpy(b).to(device) if b is not None else None
                B.boda_stack_set_filters(self.handle, i, fw, fb)
                self.filters.append(fw)
                self.biases.append(fb)
            else:
                self.filters.append(None)
                self.biases.append(None)
        first = self.ops[0].shape
        self.in_shape = (first.N, first.C, first.H, first.W)
        self.out_shape = B.boda_stack_out_dims(self.handle, len(self.ops) - 1)
        self.out = torch.empty(self.out_shape, dtype=torch.float32, device=device)
        torch.cuda.synchronize()

    def describe(self) -> List[str]:
        return [B.boda_stack_describe(self.handle, i) for i in range(len(self.ops))]

    def kernels_per_forward(self) -> int:
        return B.boda_stack_kernels_per_fwd(self.handle)

    def forward(self, x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """One graph launch on the current stream (the graph is captured on the first call)."""
        out = self.out if out is None else out
        B.boda_stack_fwd(self.handle, x, out)
        return out

    def forward_eager(self, x: torch.Tensor, events=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Kernel-by-kernel launches; events = flat list of 3 * n_ops CUDA events for per-layer timing."""
        out = self.out if out is None else out
        B.boda_stack_fwd_eager(self.handle, x, out, None, events)
        return out

    def run_op(self, i: int, x: Optional[torch.Tensor] = None) -> None:
        """Re-runs op i alone on the activations of the last forward pass (timing aid)."""
        B.boda_stack_run_op(self.handle, i, x, self.out)

    def forward_host(self, x_host: torch.Tensor, out_host: torch.Tensor) -> None:
        """Host buffers in and out (pinned for asynchronous copies); returns after the result has landed."""
        B.boda_stack_fwd_host(self.handle, x_host, out_host)

    def layer_output(self, i: int) -> Optional[torch.Tensor]:
        """NCHW copy of the activation op i wrote during the last forward pass; None for a convolution whose
        max-pool runs inside its epilogue (its own output is never materialised, only the pooled one)."""
        if i == len(self.ops) - 1:
            return self.out.clone()
        shape = B.boda_stack_out_dims(self.handle, i)
        dst = torch.empty(shape, dtype=torch.float32, device=self.out.device)
        try:
            B.boda_stack_copy_layer_output(self.handle, i, dst)
        except B.BodaError as e:
            if e.status == B.BODA_ERR_UNSUPPORTED:
                return None
            raise
        torch.cuda.synchronize()
        return dst

    def close(self) -> None:
        if self.handle:
            B.boda_stack_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
