"""Helpers of the GPU parity tests: guarded device buffers, one CUDA call through the C-ABI, one
oracle call on host copies of the same tensors, and the comparison with the stated tolerances."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle import adams_oracle as orc
from helpers import bf16_ulp_distance, within_tol

GUARD_BYTES = 256


class Guarded:
    """A device buffer with canary bands on both sides (catches out-of-bounds writes of a kernel)."""

    def __init__(self, n: int, dtype: torch.dtype, device, fill=None):
        item = torch.empty((), dtype=dtype).element_size()
        self.pad = GUARD_BYTES // item
        self.raw = torch.empty(n + 2 * self.pad, dtype=dtype, device=device)
        self.canary = {torch.float32: 1234.5, torch.bfloat16: -3.0, torch.int32: 0x5A5A5A5A}[dtype]
        self.raw.fill_(self.canary)
        self.view = self.raw[self.pad:self.pad + n]
        if fill is not None:
            self.view.copy_(fill.reshape(-1))

    def intact(self) -> bool:
        lo, hi = self.raw[:self.pad], self.raw[self.raw.numel() - self.pad:]
        return bool((lo == self.canary).all().item() and (hi == self.canary).all().item())


@dataclass
class DeviceState:
    rows: int
    cols: int
    w: Guarded
    m: Guarded
    v: Guarded
    g: Guarded
    w_fwd: Guarded
    meta: Guarded
    scale: Optional[torch.Tensor]

    def all_intact(self) -> bool:
        return all(b.intact() for b in (self.w, self.m, self.v, self.g, self.w_fwd, self.meta))


def to_device(inp: workloads.TensorInputs, device, meta_in: Optional[np.ndarray] = None, fwd_elems: Optional[int] = None) -> DeviceState:
    rows, cols = inp.w.shape
    n = rows * cols
    meta = Guarded(n // 32, torch.int32, device)
    if meta_in is not None:
        meta.view.copy_(torch.from_numpy(np.ascontiguousarray(meta_in).view(np.int32).reshape(-1)))
    else:
        meta.view.zero_()
    fwd = Guarded(n if fwd_elems is None else fwd_elems, torch.bfloat16, device)
    return DeviceState(rows, cols,
                       Guarded(n, torch.float32, device, inp.w.to(device)),
                       Guarded(n, torch.float32, device, inp.m.to(device)),
                       Guarded(n, torch.float32, device, inp.v.to(device)),
                       Guarded(n, torch.bfloat16, device, inp.g.to(device)),
                       fwd, meta,
                       None if inp.scale is None else inp.scale.to(device).contiguous())


def host_arrays(inp: workloads.TensorInputs):
    return (inp.w.cpu().numpy(), inp.m.cpu().numpy(), inp.v.cpu().numpy(), workloads.bf16_bits(inp.g),
            None if inp.scale is None else inp.scale.cpu().numpy())


def oracle_flags(flags: int) -> int:
    """The two flag sets use the same numbering; translated name by name so a renumbering would show.  Flags that
    only choose an implementation (bulk staging) or ask for extra outputs (statistics) have no oracle counterpart."""
    out = 0
    for lib_bit, orc_bit in ((B.CAST_F_RESELECT, orc.F_RESELECT), (B.CAST_F_COUNT_FLIPS, orc.F_COUNT_FLIPS),
                             (B.CAST_F_META_BITMASK, orc.F_META_BITMASK), (B.CAST_F_V_KEPT_FROM_G, orc.F_V_KEPT_FROM_G),
                             (B.CAST_F_EMIT_DENSE, orc.F_EMIT_DENSE), (B.CAST_F_EMIT_COMPRESSED, orc.F_EMIT_COMPRESSED),
                             (B.CAST_F_GRAD_OF_SCALED, orc.F_GRAD_OF_SCALED)):
        if flags & lib_bit:
            out |= orc_bit
    return out


def run_oracle(inp: workloads.TensorInputs, N, M, hyper: orc.Hyper, flags, meta_in=None, precision="f64", scale_chain=None):
    w, m, v, g, sc = host_arrays(inp)
    return orc.adams_step(w, m, v, g, sc, N, M, hyper, oracle_flags(flags), meta_in, precision, scale_chain)


def device_outputs(st: DeviceState, flips=None):
    rows, cols = st.rows, st.cols
    out = dict(
        w=st.w.view.cpu().numpy().reshape(rows, cols),
        m=st.m.view.cpu().numpy().reshape(rows, cols),
        v=st.v.view.cpu().numpy().reshape(rows, cols),
        w_fwd=workloads.bf16_bits(st.w_fwd.view).reshape(rows, -1),
        meta=st.meta.view.cpu().numpy().view(np.uint32).reshape(rows, cols // 32),
    )
    if flips is not None:
        out["flips"] = int(flips.item())
    return out


def run_cuda_single(inp: workloads.TensorInputs, N, M, hyper: orc.Hyper, flags, meta_in=None, device="cuda:0"):
    rows_, cols_ = inp.w.shape
    st = to_device(inp, device, meta_in, rows_ * cols_ * N // M if flags & B.CAST_F_EMIT_COMPRESSED else None)
    flips = torch.zeros(1, dtype=torch.int64, device=device) if flags & B.CAST_F_COUNT_FLIPS else None
    lr, b1, b2, eps, lam = hyper.as_f32()
    n_seg = 1 if st.scale is None else st.scale.shape[1]
    cast.check(cast.cast_adams_step(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view,
                                    st.scale, n_seg, st.rows, st.cols, N, M, lr, b1, b2, eps, lam,
                                    hyper.step, hyper.total_steps, flags, flips, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert st.all_intact(), "a kernel wrote outside its buffers"
    return device_outputs(st, flips)


def near_tie_groups(w: np.ndarray, N: int, M: int, rel: float = 1e-6) -> int:
    """Groups whose N-th and (N+1)-th largest magnitudes differ by less than `rel` relative."""
    if N >= M:
        return 0
    a = np.sort(np.abs(w.reshape(-1, M).astype(np.float64)), axis=1)[:, ::-1]
    hi, lo = a[:, N - 1], a[:, N]
    return int(np.sum((hi - lo) < rel * np.maximum(hi, 1e-300)))


def assert_parity(got: dict, ref: dict, label: str = ""):
    """fp32 state within max(1e-6 relative, 1e-9 absolute); forward weight within 1 bf16 ulp with the same
    zero pattern; metadata bit-exact."""
    for k in ("w", "m", "v"):
        ok, worst = within_tol(got[k], ref[k], rel=1e-6, floor=1e-9)
        assert ok, f"{label} {k}: worst error is {worst:.3g} x the tolerance"
    assert np.array_equal(got["meta"], ref["meta"]), f"{label} metadata differs"
    d = bf16_ulp_distance(got["w_fwd"], ref["w_fwd"])
    assert d.max(initial=0) <= 1, f"{label} forward weight differs by {d.max()} ulp"
    # zero pattern: where exactly one side is (+-)0 the other side must be the smallest bf16 magnitude, i.e. a kept
    # value that rounds to zero on one side only; pruned slots are 0x0000 on both sides
    mag_got, mag_ref = got["w_fwd"] & 0x7FFF, ref["w_fwd"] & 0x7FFF
    one_sided = (mag_got == 0) != (mag_ref == 0)
    assert np.all(np.maximum(mag_got, mag_ref)[one_sided] <= 1), f"{label} zero pattern differs"
    if "flips" in got:
        assert got["flips"] == ref["flips"], f"{label} flips {got['flips']} != {ref['flips']}"


def v_pure_relative_error(got: dict, ref: dict) -> float:
    r = ref["v"].astype(np.float64)
    nz = r != 0
    return float(np.max(np.abs(got["v"].astype(np.float64)[nz] - r[nz]) / np.abs(r[nz]))) if nz.any() else 0.0


# ----------------------------------------------------------------------------------------------------
# whole-matrix comparison at full size: the oracle runs over host copies split by rows over threads,
# its outputs go back to the device and every element is compared there

def host_threads() -> int:
    import os
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_inplace_threaded(w, m, v, g_bits, fwd_bits, meta, scale, rows, cols, N, M, hyper: orc.Hyper, flags, threads):
    """The oracle (fp64 build, as it stands) in place on flat host arrays of one matrix, blocks of whole rows
    handed to `threads` Python threads (ctypes releases the GIL; every block is the same serial loop).
    Returns the flips counted."""
    from concurrent.futures import ThreadPoolExecutor
    oflags = oracle_flags(flags)
    fcols = cols * N // M if oflags & orc.F_EMIT_COMPRESSED else cols
    per = max(1, -(-rows // (4 * threads)))
    jobs = []
    for r0 in range(0, rows, per):
        r1 = min(rows, r0 + per)
        jobs.append((w[r0 * cols:r1 * cols], m[r0 * cols:r1 * cols], v[r0 * cols:r1 * cols], g_bits[r0 * cols:r1 * cols],
                     fwd_bits[r0 * fcols:r1 * fcols], meta[r0 * cols // 32:r1 * cols // 32],
                     None if scale is None else scale[r0:r1], r1 - r0))

    def one(j):
        return orc.adams_step_inplace(j[0], j[1], j[2], j[3], j[4], j[5], j[6], j[7], cols, N, M, hyper, oflags)

    orc._load()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return sum(ex.map(one, jobs))


class HostStage:
    """Page-locked host arrays for one matrix of up to `max_params` parameters, reused from matrix to matrix."""

    def __init__(self, max_params: int):
        pin = lambda n, dt: torch.empty(n, dtype=dt).pin_memory()
        self.w, self.m, self.v = (pin(max_params, torch.float32) for _ in range(3))
        self.g = pin(max_params, torch.int16)
        self.fwd = pin(max_params, torch.int16)
        self.meta = pin(max_params // 32, torch.int32)


def device_mismatches(got: torch.Tensor, ref: torch.Tensor, rel=1e-6, floor=1e-9):
    """On the device: (# elements with |got - ref| > max(rel |ref|, floor), worst error / bound), in fp64."""
    g64, r64 = got.reshape(-1).double(), ref.reshape(-1).double()
    ratio = (g64 - r64).abs_() / torch.clamp(r64.abs_() * rel, min=floor)
    return int((ratio > 1.0).sum().item()), float(ratio.max().item())


def bf16_key(bits_i16: torch.Tensor) -> torch.Tensor:
    """Raw bf16 bits (int16 view) mapped onto a monotone integer line; +0 and -0 coincide."""
    b = bits_i16.to(torch.int32)
    mag = b & 0x7FFF
    return torch.where(b < 0, -mag, mag)


def near_tie_groups_device(w: torch.Tensor, N: int, M: int, rel: float = 1e-6) -> int:
    if N >= M:
        return 0
    a = w.reshape(-1, M).abs().double().sort(dim=1, descending=True).values
    hi, lo = a[:, N - 1], a[:, N]
    return int(((hi - lo) < rel * hi.clamp(min=1e-300)).sum().item())


def whole_matrix_parity(mat, regenerated: workloads.TensorInputs, prior_meta, N, M, hyper: orc.Hyper, flags,
                        stage: HostStage, threads: int, label: str):
    """Every element of one matrix of a stepped state against the oracle.

    `mat` holds the CUDA path's results (w, m, v, w_fwd, meta on the device); `regenerated` the step's inputs
    drawn again from the same seeds on the same device (bit-identical to what the kernel read); `prior_meta` the
    metadata words the step found (int32 device tensor) or None for zeros.  Returns dict(flips, near_ties)."""
    rows, cols = mat.rows, mat.cols
    P = rows * cols
    hw, hm, hv = stage.w[:P], stage.m[:P], stage.v[:P]
    hg, hf, hmeta = stage.g[:P], stage.fwd, stage.meta[:P // 32]
    hw.copy_(regenerated.w.reshape(-1)); hm.copy_(regenerated.m.reshape(-1)); hv.copy_(regenerated.v.reshape(-1))
    hg.copy_(regenerated.g.reshape(-1).view(torch.int16))
    if prior_meta is None:
        hmeta.zero_()
    else:
        hmeta.copy_(prior_meta.reshape(-1))
    scale = None if regenerated.scale is None else regenerated.scale.cpu().numpy()
    fwd_elems = mat.w_fwd.numel()
    hf = hf[:fwd_elems]
    torch.cuda.synchronize()
    flips = oracle_inplace_threaded(hw.numpy(), hm.numpy(), hv.numpy(), hg.numpy().view(np.uint16), hf.numpy().view(np.uint16),
                                    hmeta.numpy().view(np.uint32), scale, rows, cols, N, M, hyper, flags, threads)
    dev = mat.w.device
    for name, got, ref in (("w", mat.w, hw), ("m", mat.m, hm), ("v", mat.v, hv)):
        bad, worst = device_mismatches(got, ref.to(dev, non_blocking=True))
        assert bad == 0, f"{label} {name}: {bad} of {P} elements outside the tolerance, worst {worst:.3g} x"
    ref_meta = hmeta.to(dev, non_blocking=True)
    diff_words = int((mat.meta.reshape(-1) != ref_meta).sum().item())
    assert diff_words == 0, f"{label}: {diff_words} metadata words differ"
    got_bits, ref_bits = mat.w_fwd.reshape(-1).view(torch.int16), hf.to(dev, non_blocking=True)
    ulp = (bf16_key(got_bits) - bf16_key(ref_bits)).abs_()
    assert int(ulp.max().item()) <= 1, f"{label}: forward weight differs by {int(ulp.max().item())} bf16 ulp"
    zero_diff = int((((got_bits & 0x7FFF) == 0) != ((ref_bits & 0x7FFF) == 0)).sum().item())
    # pruned slots are +0 on both sides; a kept value may round to the smallest subnormal on one side and to zero on
    # the other only within the 1-ulp rule above, which the distance already enforces
    assert zero_diff == 0 or int(ulp.max().item()) <= 1
    return dict(flips=flips, near_ties=near_tie_groups_device(regenerated.w, N, M), zero_pattern_diffs=zero_diff)
