"""A chain of convolution and pooling layers driven through the C ABI (layer i+1 eats layer i's output).

Host-side orchestration only: it creates one plan per convolution, keeps the activations in device
tensors and issues the library calls in order on one stream.  No arithmetic happens here.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B
from .workloads import StackOp


class ConvStack:
    def __init__(self, ops: Sequence[StackOp], params: Sequence[Tuple], math: int = B.BODA_MATH_AUTO,
                 tune: int = 0, device: str = "cuda"):
        """ops: conv / pool descriptors; params: per conv layer (filters, bias) as numpy fp32 arrays."""
        self.ops = list(ops)
        self.device = device
        self.plans: List[Optional[B.ConvPlan]] = []
        self.filters: List[Optional[torch.Tensor]] = []
        self.biases: List[Optional[torch.Tensor]] = []
        self.outputs: List[torch.Tensor] = []
        it = iter(params)
        shape_nchw = None
        ws_bytes = 0
        for op in self.ops:
            if op.kind == "conv":
                s = op.shape
                w, b = next(it)
                plan = B.ConvPlan(s.as_tuple(), math=math, tune=tune)
                fw = torch.from_numpy(w).to(device)
                plan.bind_filters(fw)
                self.plans.append(plan)
                self.filters.append(fw)
                self.biases.append(torch.from_numpy(b).to(device) if b is not None else None)
                shape_nchw = plan.out_shape
                if shape_nchw is None:
                    raise ValueError("bad conv shape")
            else:
                N, C, H, W = shape_nchw
                shape_nchw = (N, C, B.boda_conv_out_dim(H, op.ksz, op.stride, 0), B.boda_conv_out_dim(W, op.ksz, op.stride, 0))
                self.plans.append(None)
                self.filters.append(None)
                self.biases.append(None)
            self.outputs.append(torch.empty(shape_nchw, dtype=torch.float32, device=device))
        first = self.ops[0].shape
        self.in_shape = (first.N, first.C, first.H, first.W)
        self.out_shape = tuple(self.outputs[-1].shape)
        self.staging_in = torch.empty(self.in_shape, dtype=torch.float32, device=device)
        torch.cuda.synchronize()

    def describe(self) -> List[str]:
        return [p.describe() if p is not None else "maxpool" for p in self.plans]

    def forward(self, x: torch.Tensor, events=None) -> torch.Tensor:
        """Runs every layer on the current stream.  events: optional list of (start, end) CUDA event pairs,
        one per op, recorded around that op's launches."""
        cur = x
        for i, op in enumerate(self.ops):
            if events is not None:
                events[i][0].record()
            out = self.outputs[i]
            if op.kind == "conv":
                B.boda_conv_fwd_planned(self.plans[i].handle, cur, self.filters[i], self.biases[i], out,
                                        self.plans[i].workspace)
            else:
                N, C, H, W = cur.shape
                B.boda_maxpool_fwd(cur, out, N, C, H, W, op.ksz, op.stride)
            if events is not None:
                events[i][1].record()
            cur = out
        return cur

    def forward_host(self, x_host: torch.Tensor, out_host: torch.Tensor) -> None:
        """Host buffers in and out (pinned for asynchronous copies); returns after the result has landed."""
        self.staging_in.copy_(x_host, non_blocking=True)
        y = self.forward(self.staging_in)
        out_host.copy_(y, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    def close(self) -> None:
        for p in self.plans:
            if p is not None:
                p.close()
