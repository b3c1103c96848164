"""Seeded synthetic inputs and the layer-shape lists of the benchmark workloads.

This module holds NO arithmetic of the method: it only names shapes and draws
random tensors.  Both the CUDA path and the CPU oracle are fed from here, so
that they see bit-identical inputs (a tensor is drawn once, on one device, and
copied to wherever the other side needs it).

The tensors stand in for the linear layers of the models the paper trains
(OPT-125M / GPT-2 small: d=768, ffn=3072; LLaMA2-7B: d=4096, ffn=11008;
LLaMA2-13B: d=5120, ffn=13824).  Weights are stored [out_features, in_features]
row-major; the N:M groups run along in_features (Eq. 3).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch

Shape = Tuple[int, int]

W_STD = 0.02      # master weights  ~ N(0, 0.02^2)
G_STD = 1e-3      # gradients       ~ N(0, 1e-6), rounded to bf16
M_STD = 1e-4      # first moments   ~ N(0, 1e-8)
VZ_STD = 1e-3     # second moments  = z^2, z ~ N(0, 1e-6)

SCALE_SEGMENTS = 2   # n = 2 row segments per scale vector (the paper's setting, Sec. 6.1)


def decoder_linear_shapes(n_layers: int, d: int, ffn: int, gated: bool) -> List[Shape]:
    """[rows, cols] of every prunable linear weight of a decoder stack."""
    per_layer: List[Shape] = [(d, d)] * 4
    if gated:                      # LLaMA: gate, up: ffn x d; down: d x ffn
        per_layer += [(ffn, d), (ffn, d), (d, ffn)]
    else:                          # shapes exactly as the workload list writes them
        per_layer += [(d, ffn), (ffn, d)]
    return per_layer * n_layers


@dataclass(frozen=True)
class Workload:
    name: str
    shapes: Tuple[Shape, ...]
    total_steps: int              # T of alpha_t = t/T (Table 11 step counts)
    note: str = ""
    layer_matrices: int = 0       # matrices per decoder layer (0: not a layered workload)
    resident_layers: int = 0      # > 0: only this many layers of state are resident; the layers are stepped
                                  # one call per layer, layer L in slot L mod resident_layers

    @property
    def n_params(self) -> int:
        return sum(r * c for r, c in self.shapes)


def workload(name: str) -> Workload:
    if name == "opt125m_fc2":
        return Workload(name, ((3072, 768),), 30000, "one 3072x768 matrix")
    if name == "decoder_d768_12l":
        return Workload(name, tuple(decoder_linear_shapes(12, 768, 3072, gated=False)), 30000,
                        "12 layers, d=768, ffn=3072, 72 matrices")
    if name == "llama2_7b":
        return Workload(name, tuple(decoder_linear_shapes(32, 4096, 11008, gated=True)), 7500,
                        "32 layers, d=4096, ffn=11008, 224 matrices")
    if name == "llama2_7b_layer":
        return Workload(name, tuple(decoder_linear_shapes(1, 4096, 11008, gated=True)), 7500,
                        "1 layer of LLaMA2-7B, 7 matrices")
    if name == "llama2_13b_layer":
        return Workload(name, tuple(decoder_linear_shapes(1, 5120, 13824, gated=True)), 7500,
                        "1 layer of LLaMA2-13B, 7 matrices")
    if name == "llama2_13b":
        return Workload(name, tuple(decoder_linear_shapes(40, 5120, 13824, gated=True)), 7500,
                        "40 layers, d=5120, ffn=13824, 280 matrices; per-layer calls on 2 streams over 10 resident layer slots",
                        layer_matrices=7, resident_layers=10)
    raise KeyError(name)


def tensor_seed(seed: int, tensor_index: int, which: int) -> int:
    """One generator seed per (run seed, tensor, field); which: 0 w, 1 g, 2 m, 3 v, 4 scale."""
    return seed * (1 << 20) + tensor_index * 8 + which


def _randn(shape, seed: int, device) -> torch.Tensor:
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


@dataclass
class TensorInputs:
    w: torch.Tensor                 # fp32 [rows, cols]
    g: torch.Tensor                 # bf16 [rows, cols]
    m: torch.Tensor                 # fp32 [rows, cols]
    v: torch.Tensor                 # fp32 [rows, cols], >= 0
    scale: Optional[torch.Tensor]   # fp32 [rows, n] or None (all ones)


def gen_tensor_inputs(rows: int, cols: int, seed: int = 0, tensor_index: int = 0,
                      device="cpu", scale_mode: str = "ones") -> TensorInputs:
    """Draw the state and gradient of one matrix.

    scale_mode: "none" (no scale tensor), "ones" (all 1, the paper's initial
    value) or "jitter" (1 + 0.1 U(0,1), used by parity tests so that a wrong
    segment index shows)."""
    shape = (rows, cols)
    w = _randn(shape, tensor_seed(seed, tensor_index, 0), device).mul_(W_STD)
    g = _randn(shape, tensor_seed(seed, tensor_index, 1), device).mul_(G_STD).to(torch.bfloat16)
    m = _randn(shape, tensor_seed(seed, tensor_index, 2), device).mul_(M_STD)
    z = _randn(shape, tensor_seed(seed, tensor_index, 3), device).mul_(VZ_STD)
    v = z.mul_(z)
    scale = None
    if scale_mode == "ones":
        scale = torch.ones((rows, SCALE_SEGMENTS), dtype=torch.float32, device=device)
    elif scale_mode == "jitter":
        gen = torch.Generator(device=device)
        gen.manual_seed(tensor_seed(seed, tensor_index, 4))
        u = torch.rand((rows, SCALE_SEGMENTS), generator=gen, device=device, dtype=torch.float32)
        scale = 1.0 + 0.1 * u
    elif scale_mode != "none":
        raise ValueError(scale_mode)
    return TensorInputs(w=w, g=g, m=m, v=v, scale=scale)


def gen_gradient(rows: int, cols: int, seed: int, tensor_index: int, step: int, device="cpu") -> torch.Tensor:
    """A fresh bf16 gradient for a later step of a multi-step run."""
    s = tensor_seed(seed, tensor_index, 1) + (step << 40)
    return _randn((rows, cols), s, device).mul_(G_STD).to(torch.bfloat16)


def bf16_bits(t: torch.Tensor):
    """Raw bits of a bf16 tensor as a numpy uint16 array (host copy)."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
