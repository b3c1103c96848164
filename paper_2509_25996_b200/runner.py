"""Device-resident optimizer state for a list of matrices, stepped through the multi-tensor plan.

This is plumbing around the C-ABI (allocation with torch, one plan, one launch per step);
every arithmetic step runs in the CUDA library.
"""
from __future__ import annotations

import ctypes
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
    scale_grad: Optional[torch.Tensor] = None      # fp32 [rows, n]; with a learned scale
    scale_m: Optional[torch.Tensor] = None         # Adam moments of the scale
    scale_v: Optional[torch.Tensor] = None
    meta_ref: Optional[torch.Tensor] = None        # int32 [rows, cols/32]; reference mask of the App. C statistics
    scale_chain: Optional[torch.Tensor] = None     # fp32 [rows, n]; the scale the last emission used (with a learned scale)


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
                 device="cuda:0", scale_mode: str = "ones", first_tensor_index: int = 0, compressed: bool = False,
                 learned_scale: bool = False, reference_masks: bool = False):
        """compressed: the forward-weight buffers hold only the kept entries ([rows, cols*N/M]); every step of
        this state then carries CAST_F_EMIT_COMPRESSED.
        learned_scale: every matrix gets a scale-gradient buffer (filled by steps that carry
        CAST_F_GRAD_OF_SCALED) and Adam moments for its scale; scale_step() then trains the scales.
        reference_masks: every matrix gets a second metadata buffer (zeros until the caller fills it, e.g. with
        the initial mask), against which steps that carry CAST_F_MASK_STATS count ||M_t - M_ref||_0; the sums
        land in self.stats (the plan is created with CAST_F_MASK_STATS)."""
        self.device = torch.device(device)
        self.N, self.M = N, M
        self.compressed = compressed
        self.seed, self.scale_mode, self.first_tensor_index = seed, scale_mode, first_tensor_index
        self.reference_masks = reference_masks
        self.plan = None
        self.mats: List[MatrixState] = []
        for i, (rows, cols) in enumerate(shapes):
            inp = workloads.gen_tensor_inputs(rows, cols, seed=seed, tensor_index=first_tensor_index + i,
                                              device=self.device, scale_mode=scale_mode)
            self.mats.append(MatrixState(
                rows, cols, inp.w, inp.m, inp.v, inp.g,
                torch.empty((rows, cols * N // M if compressed else cols), dtype=torch.bfloat16, device=self.device),
                torch.zeros((rows, cols // 32), dtype=torch.int32, device=self.device),
                inp.scale))
            if learned_scale:
                if inp.scale is None:
                    raise ValueError("a learned scale needs a scale tensor")
                mat = self.mats[-1]
                mat.scale_grad = torch.zeros_like(inp.scale)
                mat.scale_m = torch.zeros_like(inp.scale)
                mat.scale_v = torch.zeros_like(inp.scale)
                mat.scale_chain = inp.scale.clone()
            if reference_masks:
                self.mats[-1].meta_ref = torch.zeros_like(self.mats[-1].meta)
        self.n_params = sum(s.rows * s.cols for s in self.mats)
        self.flips = torch.zeros(1, dtype=torch.int64, device=self.device)
        self.stats = torch.zeros(ctypes.sizeof(B.cast_mask_stats_t), dtype=torch.uint8, device=self.device)
        self._make_plan()

    def _make_plan(self) -> None:
        tensors = [B.make_tensor(s.w, s.m, s.v, s.g, s.w_fwd, s.meta, s.scale,
                                 1 if s.scale is None else s.scale.shape[1], s.rows, s.cols, s.scale_grad, s.meta_ref, s.scale_chain)
                   for s in self.mats]
        rc, self.plan = B.cast_plan_create_ex(tensors, self.N, self.M, (B.CAST_F_EMIT_COMPRESSED if self.compressed else 0) |
                                              (B.CAST_F_MASK_STATS if self.reference_masks else 0))
        B.check(rc)

    def set_nm(self, N: int, M: int) -> None:
        """Another N:M pattern over the same buffers (a new plan; the state itself is not touched)."""
        if self.compressed:
            raise ValueError("the compressed forward-weight buffers are sized for one N:M")
        self.close()
        self.N, self.M = N, M
        self._make_plan()

    def reset(self) -> None:
        """Draws the initial state again, from the same seeds, into the existing buffers (metadata zeroed)."""
        for i, s in enumerate(self.mats):
            inp = workloads.gen_tensor_inputs(s.rows, s.cols, seed=self.seed, tensor_index=self.first_tensor_index + i,
                                              device=self.device, scale_mode=self.scale_mode)
            s.w.copy_(inp.w); s.m.copy_(inp.m); s.v.copy_(inp.v); s.g.copy_(inp.g)
            if s.scale is not None:
                s.scale.copy_(inp.scale)
            s.meta.zero_()
            del inp
        self.flips.zero_()

    def fresh_gradients(self, step: int) -> None:
        """A new seeded gradient for every matrix (what backpropagation would deliver at iteration `step`)."""
        for i, s in enumerate(self.mats):
            s.g.copy_(workloads.gen_gradient(s.rows, s.cols, self.seed, self.first_tensor_index + i, step, device=self.device))

    def step(self, hyper: Hyper, flags: int, stream=None) -> None:
        """One AdamS iteration over every matrix (asynchronous on `stream` or the current stream)."""
        if self.compressed:
            flags |= B.CAST_F_EMIT_COMPRESSED
        h = B.make_hyper(hyper.lr, hyper.beta1, hyper.beta2, hyper.eps, hyper.l1_coeff,
                         hyper.step, hyper.total_steps, flags)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        flips = self.flips if flags & B.CAST_F_COUNT_FLIPS else None
        if flags & B.CAST_F_MASK_STATS:
            B.check(B.cast_plan_step_stats(self.plan, h, flips, self.stats, s))
        else:
            B.check(B.cast_plan_step(self.plan, h, flips, s))

    def read_stats(self) -> "B.cast_mask_stats_t":
        """Host copy of the statistics accumulator (synchronises)."""
        return B.cast_mask_stats_t.from_buffer_copy(self.stats.cpu().numpy().tobytes())

    def scale_step(self, lr: float, hyper: Hyper, stream=None) -> None:
        """Adam step of every scale matrix from the accumulated scale gradients (which it clears), one launch."""
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        B.check(B.cast_plan_scale_adam_step(self.plan, [m.scale_m for m in self.mats], [m.scale_v for m in self.mats],
                                            lr, hyper.beta1, hyper.beta2, hyper.eps, hyper.step, True, s))

    def close(self) -> None:
        if self.plan is not None:
            B.check(B.cast_plan_destroy(self.plan))
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class StreamedModelState:
    """A model too large to keep resident: `n_slots` layers of state stay on the GPU and the `n_layers`
    layers are stepped one plan call per layer, layer L in slot L mod n_slots, the calls alternating over
    `n_streams` CUDA streams so that the tail of one layer's grid overlaps the head of the next.

    Two calls on one slot must not overlap (they update the same state): n_slots must be a multiple of
    n_streams, so that a slot is always stepped on the same stream and its calls are ordered by it."""

    def __init__(self, layer_shapes: Sequence[Tuple[int, int]], n_layers: int, n_slots: int, n_streams: int = 2,
                 N: int = 2, M: int = 4, seed: int = 0, device="cuda:0", scale_mode: str = "ones"):
        if n_slots % n_streams != 0:
            raise ValueError("n_slots must be a multiple of n_streams")
        self.device = torch.device(device)
        self.n_layers = n_layers
        per_layer = len(layer_shapes)
        self.slots = [DeviceModelState(layer_shapes, N, M, seed=seed, device=device, scale_mode=scale_mode,
                                       first_tensor_index=i * per_layer) for i in range(min(n_slots, n_layers))]
        self.streams = [torch.cuda.Stream(device=self.device) for _ in range(n_streams)]
        self.n_params = n_layers * self.slots[0].n_params
        self._done = [torch.cuda.Event() for _ in range(n_streams)]

    def step(self, hyper: Hyper, flags: int, stream=None, after_layer=None) -> None:
        """One AdamS iteration over all layers.  Work is ordered after what `stream` (default: the current
        stream) has queued so far, and `stream` waits for it at the end, so the caller can bracket steps with
        events on that one stream.  `after_layer(layer, slot_index, cuda_stream)`, if given, is called after
        each layer's launch has been queued; what it queues on that stream runs between this visit of the slot
        and the next one (used to copy a slot's state out between its visits)."""
        cur = stream if stream is not None else torch.cuda.current_stream(self.device)
        start = torch.cuda.Event()
        start.record(cur)
        for s in self.streams:
            s.wait_event(start)
        for layer in range(self.n_layers):
            slot, side = layer % len(self.slots), self.streams[layer % len(self.streams)]
            self.slots[slot].step(hyper, flags, side)
            if after_layer is not None:
                after_layer(layer, slot, side)
        for s, ev in zip(self.streams, self._done):
            ev.record(s)
            cur.wait_event(ev)

    @property
    def flips(self) -> torch.Tensor:
        return sum(s.flips for s in self.slots)

    def close(self) -> None:
        for s in self.slots:
            s.close()
