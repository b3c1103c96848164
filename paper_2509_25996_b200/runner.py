"""Device-resident optimizer state for a list of matrices, stepped through the multi-tensor plan.

This is plumbing around the C-ABI (allocation with torch, one plan, one launch per step);
every arithmetic step runs in the CUDA library.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B
from . import workloads


@dataclass
class MatrixState:
    rows: int
    cols: int
    w: torch.Tensor
    m: torch.Tensor
    v: torch.Tensor
    g: torch.Tensor
    w_fwd: torch.Tensor
    meta: torch.Tensor                 # int32 [rows, cols/32]
    scale: Optional[torch.Tensor]


@dataclass
class Hyper:
    lr: float = 1e-4
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    l1_coeff: float = 1e-3
    step: int = 1000
    total_steps: int = 30000


class DeviceModelState:
    """All prunable matrices of a model on one GPU plus the plan that steps them in one launch."""

    def __init__(self, shapes: Sequence[Tuple[int, int]], N: int = 2, M: int = 4, seed: int = 0,
                 device="cuda:0", scale_mode: str = "ones", first_tensor_index: int = 0):
        self.device = torch.device(device)
        self.N, self.M = N, M
        self.mats: List[MatrixState] = []
        for i, (rows, cols) in enumerate(shapes):
            inp = workloads.gen_tensor_inputs(rows, cols, seed=seed, tensor_index=first_tensor_index + i,
                                              device=self.device, scale_mode=scale_mode)
            self.mats.append(MatrixState(
                rows, cols, inp.w, inp.m, inp.v, inp.g,
                torch.empty((rows, cols), dtype=torch.bfloat16, device=self.device),
                torch.zeros((rows, cols // 32), dtype=torch.int32, device=self.device),
                inp.scale))
        self.n_params = sum(s.rows * s.cols for s in self.mats)
        self.flips = torch.zeros(1, dtype=torch.int64, device=self.device)
        tensors = [B.make_tensor(s.w, s.m, s.v, s.g, s.w_fwd, s.meta, s.scale,
                                 1 if s.scale is None else s.scale.shape[1], s.rows, s.cols) for s in self.mats]
        rc, self.plan = B.cast_plan_create(tensors, N, M)
        B.check(rc)

    def step(self, hyper: Hyper, flags: int, stream=None) -> None:
        """One AdamS iteration over every matrix (asynchronous on `stream` or the current stream)."""
        h = B.make_hyper(hyper.lr, hyper.beta1, hyper.beta2, hyper.eps, hyper.l1_coeff,
                         hyper.step, hyper.total_steps, flags)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        B.check(B.cast_plan_step(self.plan, h, self.flips if flags & B.CAST_F_COUNT_FLIPS else None, s))

    def close(self) -> None:
        if self.plan is not None:
            B.check(B.cast_plan_destroy(self.plan))
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
