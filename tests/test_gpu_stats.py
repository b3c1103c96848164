"""cast_mask_stats (App. C statistics) on the GPU against the CPU oracle: mask differences bit-exact, the two
magnitude sums within 1e-12 relative (both sides add exactly converted |w| in fp64; only the order differs)."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle import adams_oracle as orc
import gpu_util as U

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RS, BM = B.CAST_F_RESELECT, B.CAST_F_META_BITMASK


def read_stats(buf: torch.Tensor):
    raw = buf.cpu().numpy().tobytes()
    s = B.cast_mask_stats_t.from_buffer_copy(raw)
    return dict(flips=int(s.mask_diff), kept_abs=float(s.kept_abs_sum), total_abs=float(s.total_abs_sum), reserved=int(s.reserved_))


def masks_for(rows, cols, N, M, bitmask, seed):
    enc = orc.F_META_BITMASK if bitmask else 0
    out = []
    for k in range(2):
        inp = workloads.gen_tensor_inputs(rows, cols, seed=seed + k, scale_mode="none")
        out.append(U.run_oracle(inp, N, M, orc.Hyper(), RS | (BM if bitmask else 0))["meta"])
    return out


def gpu_stats(w, meta, meta_ref, M, bitmask, stats=None):
    rows, cols = w.shape
    d_w = w.to(DEV).contiguous()
    d_meta = torch.from_numpy(meta.view(np.int32).copy()).to(DEV)
    d_ref = None if meta_ref is None else torch.from_numpy(meta_ref.view(np.int32).copy()).to(DEV)
    if stats is None:
        stats = torch.zeros(ctypes.sizeof(B.cast_mask_stats_t), dtype=torch.uint8, device=DEV)
    before = cast.cast_kernel_launch_count()
    cast.check(cast.cast_mask_stats(d_w, d_meta, d_ref, rows, cols, M, BM if bitmask else 0, stats, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + 1
    return stats


def assert_stats(got, ref, label):
    assert got["flips"] == ref["flips"], f"{label}: mask difference {got['flips']} != {ref['flips']}"
    assert got["kept_abs"] == pytest.approx(ref["kept_abs"], rel=1e-12), label
    assert got["total_abs"] == pytest.approx(ref["total_abs"], rel=1e-12), label
    assert got["reserved"] == 0


@pytest.mark.parametrize("N,M,bitmask", [(2, 4, False), (2, 4, True), (1, 4, True), (4, 8, True), (5, 16, True), (8, 32, True)])
@pytest.mark.parametrize("rows,cols", [(1, 32), (5, 96), (9, 8224), (64, 4096)])
def test_stats_match_oracle(N, M, bitmask, rows, cols):
    """From one unit to 8 tiles of 32768 parameters, with ragged batches and tiles (9 x 8224 = 2.26 tiles)."""
    meta, meta_ref = masks_for(rows, cols, N, M, bitmask, seed=70)
    w = workloads.gen_tensor_inputs(rows, cols, seed=72, scale_mode="none").w
    for ref_mask in (meta_ref, None):
        got = read_stats(gpu_stats(w, meta, ref_mask, M, bitmask))
        assert_stats(got, orc.mask_stats(w.numpy(), meta, ref_mask, M, bitmask), f"{N}:{M} {rows}x{cols} ref={ref_mask is not None}")


def test_stats_accumulate_over_matrices_and_special_values():
    """The call adds to the counters: two matrices give the model-wide sums.  Zeros of both signs, denormals and
    large magnitudes go through |w| unchanged."""
    stats = None
    want = dict(flips=0, kept_abs=0.0, total_abs=0.0)
    for i, (rows, cols) in enumerate([(7, 1056), (3, 2048)]):
        meta, meta_ref = masks_for(rows, cols, 2, 4, False, seed=80 + 2 * i)
        w = workloads.gen_tensor_inputs(rows, cols, seed=90 + i, scale_mode="none").w
        w.view(-1)[0::11] = 0.0
        w.view(-1)[1::11] = -0.0
        w.view(-1)[2::11] = 1e-41
        w.view(-1)[3::11] = -3e4
        stats = gpu_stats(w, meta, meta_ref, 4, False, stats)
        r = orc.mask_stats(w.numpy(), meta, meta_ref, 4, False)
        for k in want:
            want[k] += r[k]
    assert_stats(read_stats(stats), want, "two matrices")


def test_plan_stats_one_launch_over_mixed_shapes():
    """All matrices of a plan in one grid: ragged tiles, one-unit matrices, with and without reference masks."""
    shapes = [(1, 32), (3, 96), (64, 1056), (9, 8224), (1, 32), (33, 2048), (300, 1024)]
    states, refs, want = [], [], dict(flips=0, kept_abs=0.0, total_abs=0.0)
    want_noref = dict(flips=0, kept_abs=0.0, total_abs=0.0)
    for i, (r, c) in enumerate(shapes):
        meta, meta_ref = masks_for(r, c, 4, 8, True, seed=100 + 2 * i)
        inp = workloads.gen_tensor_inputs(r, c, seed=120 + i, scale_mode="none")
        st = U.to_device(inp, DEV, meta)
        states.append(st)
        refs.append(torch.from_numpy(meta_ref.view(np.int32).copy()).to(DEV))
        o = orc.mask_stats(inp.w.numpy(), meta, meta_ref, 8, True)
        for k in want:
            want[k] += o[k]
            want_noref[k] += o[k] if k != "flips" else 0
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, None, 1, s.rows, s.cols) for s in states]
    rc, plan = cast.cast_plan_create(tensors, 4, 8)
    cast.check(rc)
    for meta_refs, expect in ((refs, want), (None, want_noref)):
        stats = torch.zeros(32, dtype=torch.uint8, device=DEV)
        before = cast.cast_kernel_launch_count()
        cast.check(cast.cast_plan_mask_stats(plan, meta_refs, BM, stats, torch.cuda.current_stream()))
        torch.cuda.synchronize()
        assert cast.cast_kernel_launch_count() == before + 1
        assert_stats(read_stats(stats), expect, f"plan, refs={meta_refs is not None}")
    assert cast.cast_plan_mask_stats(plan, None, 0, stats, None) == B.CAST_ERR_NM          # index form needs M == 4
    assert cast.cast_plan_mask_stats(None, None, BM, stats, None) == B.CAST_ERR_PLAN
    cast.check(cast.cast_plan_destroy(plan))
    assert all(s.all_intact() for s in states)


def test_stats_after_a_step_on_one_llama_matrix():
    """A 4096 x 11008 matrix (45 M parameters, 5504 tiles): the statistics of the state the AdamS kernel leaves,
    against the mask it had before (flips of the step, counted a second way) and against the oracle."""
    rows, cols = 4096, 11008
    inp = workloads.gen_tensor_inputs(rows, cols, seed=0, tensor_index=6, device=DEV, scale_mode="ones")
    prev = torch.zeros((rows, cols // 32), dtype=torch.int32, device=DEV)
    meta = torch.zeros((rows, cols // 32), dtype=torch.int32, device=DEV)
    fwd = torch.empty((rows, cols), dtype=torch.bfloat16, device=DEV)
    h = orc.Hyper(total_steps=7500)
    lr, b1, b2, eps, lam = h.as_f32()
    st = torch.cuda.current_stream()
    # mask of the initial weights, then one step with a large learning rate so that some groups change their kept set
    cast.check(cast.cast_adams_step(inp.w.clone(), inp.m.clone(), inp.v.clone(), inp.g, fwd, prev, inp.scale, 2, rows, cols, 2, 4,
                                    0.0, b1, b2, eps, lam, h.step, h.total_steps, RS, None, st))
    meta.copy_(prev)
    flips = torch.zeros(1, dtype=torch.int64, device=DEV)
    cast.check(cast.cast_adams_step(inp.w, inp.m, inp.v, inp.g, fwd, meta, inp.scale, 2, rows, cols, 2, 4,
                                    2e-4, b1, b2, eps, lam, h.step, h.total_steps, RS, None, st))
    cast.check(cast.cast_adams_step(inp.w, inp.m, inp.v, inp.g, fwd, meta, inp.scale, 2, rows, cols, 2, 4,
                                    2e-4, b1, b2, eps, lam, h.step + 1, h.total_steps, RS | B.CAST_F_COUNT_FLIPS, flips, st))
    stats = torch.zeros(32, dtype=torch.uint8, device=DEV)
    cast.check(cast.cast_mask_stats(inp.w, meta, prev, rows, cols, 4, 0, stats, st))
    torch.cuda.synchronize()
    got = read_stats(stats)
    ref = orc.mask_stats(inp.w.cpu().numpy(), meta.cpu().numpy().view(np.uint32), prev.cpu().numpy().view(np.uint32), 4, False)
    assert_stats(got, ref, "4096x11008")
    assert got["flips"] > 0 and int(flips.item()) > 0
    # the pruned forward weight holds exactly the kept entries: its non-zeros are the mask
    assert 0.5 < got["kept_abs"] / got["total_abs"] < 1.0
