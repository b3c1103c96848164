"""The App. C statistics as an epilogue of the AdamS step (CAST_F_MASK_STATS) against the CPU oracle: the fused
step is compared with oracle_adams_step followed by oracle_mask_stats on ITS outputs.

Tolerances.  The mask difference ||M_t - M_ref||_0 is exact (the kept set is bit-exact).  The two magnitude sums
are taken over the updated weights, which the CUDA path has within max(1e-6 |w|, 1e-9) of the oracle's, so the
sums agree within 1e-6 * sum|w| + 1e-9 * n.  The summation itself is exact up to its order: against an fp64 sum
over the CUDA path's OWN updated weights (mask decoded independently of both implementations) the sums agree
within 1e-12 relative."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from paper_2509_25996_b200.runner import DeviceModelState, Hyper as RunHyper
from oracle import adams_oracle as orc
from oracle.adams_oracle import Hyper
from helpers import keep_mask_from_meta
import gpu_util as U

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RS, BM, FL, DN, ST = B.CAST_F_RESELECT, B.CAST_F_META_BITMASK, B.CAST_F_COUNT_FLIPS, B.CAST_F_EMIT_DENSE, B.CAST_F_MASK_STATS


def read_stats(buf):
    s = B.cast_mask_stats_t.from_buffer_copy(buf.cpu().numpy().tobytes())
    return dict(flips=int(s.mask_diff), kept_abs=float(s.kept_abs_sum), total_abs=float(s.total_abs_sum), reserved=int(s.reserved_))


def step_with_stats(inp, N, M, h, flags, meta_in, meta_ref):
    """One fused step of a one-matrix plan on guarded buffers; returns (outputs, statistics)."""
    st = U.to_device(inp, DEV, meta_in, inp.w.numel() * N // M if flags & B.CAST_F_EMIT_COMPRESSED else None)
    d_ref = None if meta_ref is None else torch.from_numpy(np.ascontiguousarray(meta_ref).view(np.int32).reshape(-1)).to(DEV)
    flips = torch.zeros(1, dtype=torch.int64, device=DEV) if flags & FL else None
    stats = torch.zeros(ctypes.sizeof(B.cast_mask_stats_t), dtype=torch.uint8, device=DEV)
    lr, b1, b2, eps, lam = h.as_f32()
    t = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, st.scale,
                      1 if st.scale is None else st.scale.shape[1], st.rows, st.cols, None, d_ref)
    rc, plan = B.cast_plan_create_ex([t], N, M, ST | (flags & B.CAST_F_EMIT_COMPRESSED))
    cast.check(rc)
    before = cast.cast_kernel_launch_count()
    hy = B.make_hyper(lr, b1, b2, eps, lam, h.step, h.total_steps, flags)
    cast.check(cast.cast_plan_step_stats(plan, hy, flips, stats, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + 2          # the step and the one-CTA fold of the partial sums
    assert st.all_intact()
    cast.check(cast.cast_plan_destroy(plan))
    return U.device_outputs(st, flips), read_stats(stats)


def check_stats(got_out, got_stats, ref_out, meta_ref, M, bitmask, label):
    rows, cols = ref_out["w"].shape
    want = orc.mask_stats(ref_out["w"], ref_out["meta"], meta_ref, M, bitmask)
    assert got_stats["flips"] == want["flips"], f"{label}: mask difference {got_stats['flips']} != {want['flips']}"
    n = rows * cols
    for k in ("kept_abs", "total_abs"):
        assert abs(got_stats[k] - want[k]) <= 1e-6 * want["total_abs"] + 1e-9 * n, f"{label} {k}"
    assert got_stats["reserved"] == 0
    # the summation itself: fp64 sums over the CUDA path's own updated weights, mask decoded here
    keep = keep_mask_from_meta(got_out["meta"], cols, M, bitmask)
    mag = np.abs(got_out["w"].astype(np.float64))
    assert got_stats["total_abs"] == pytest.approx(mag.sum(), rel=1e-12), label
    assert got_stats["kept_abs"] == pytest.approx(mag[keep].sum(), rel=1e-12), label


CASES = [
    (2, 4, RS | FL | DN, "the refresh step of training"),
    (2, 4, RS, "headline step"),
    (2, 4, RS | BM | FL, "2:4 as bitmask"),
    (2, 4, DN, "stored 2:4 mask, index form"),
    (2, 4, BM, "stored 2:4 mask, bitmask form"),
    (4, 8, RS | BM | FL, "4:8"),
    (1, 4, RS | BM, "1:4"),
    (3, 4, BM | DN, "stored 3:4 mask"),
    (1, 2, RS | BM, "1:2"),
    (5, 16, RS | BM | FL, "5:16"),
    (8, 32, RS | BM, "8:32"),
    (8, 32, BM, "stored 8:32 mask"),
]


@pytest.mark.parametrize("N,M,flags,what", CASES)
@pytest.mark.parametrize("rows,cols", [(1, 32), (5, 96), (7, 2080)])
def test_step_with_statistics_matches_oracle(N, M, flags, what, rows, cols):
    bitmask = bool(flags & BM)
    inp = workloads.gen_tensor_inputs(rows, cols, seed=21, tensor_index=N * 100 + M, device="cpu", scale_mode="jitter")
    if (cols // 2) % max(M, 8) != 0:
        inp.scale = None
    enc = BM if bitmask else 0
    # stored / previous mask: the kept set of other weights; reference mask: of yet other weights
    other = workloads.gen_tensor_inputs(rows, cols, seed=22, tensor_index=1, device="cpu", scale_mode="none")
    third = workloads.gen_tensor_inputs(rows, cols, seed=23, tensor_index=2, device="cpu", scale_mode="none")
    meta_in = U.run_oracle(other, N, M, Hyper(lr=0.0), RS | enc)["meta"]
    meta_ref = U.run_oracle(third, N, M, Hyper(lr=0.0), RS | enc)["meta"]
    h = Hyper()
    for ref in (meta_ref, None):
        got, stats = step_with_stats(inp, N, M, h, flags | ST, meta_in, ref)
        want = U.run_oracle(inp, N, M, h, flags, meta_in=meta_in)
        U.assert_parity(got, want, f"{what} {rows}x{cols}")
        check_stats(got, stats, want, ref, M, bitmask, f"{what} {rows}x{cols} ref={ref is not None}")
        if ref is None:
            assert stats["flips"] == 0


@pytest.mark.parametrize("flags,what", [(DN, "stored 2:4 mask, index form, dense emission")])
@pytest.mark.parametrize("rows,cols", [(1, 32), (5, 96), (7, 2080), (33, 1056)])
def test_staged_step_with_statistics_matches_oracle(flags, what, rows, cols):
    """The same on the staged access path (the sums ride on the barrier before the tile's stores), forced by flag: a
    plan takes it by itself only for launches of model size."""
    inp = workloads.gen_tensor_inputs(rows, cols, seed=24, tensor_index=7, device="cpu", scale_mode="jitter")
    if (cols // 2) % 8 != 0:
        inp.scale = None
    other = workloads.gen_tensor_inputs(rows, cols, seed=25, tensor_index=1, device="cpu", scale_mode="none")
    third = workloads.gen_tensor_inputs(rows, cols, seed=26, tensor_index=2, device="cpu", scale_mode="none")
    meta_in = U.run_oracle(other, 2, 4, Hyper(lr=0.0), RS)["meta"]
    meta_ref = U.run_oracle(third, 2, 4, Hyper(lr=0.0), RS)["meta"]
    h = Hyper()
    want = U.run_oracle(inp, 2, 4, h, flags, meta_in=meta_in)
    for ref in (meta_ref, None):
        got, stats = step_with_stats(inp, 2, 4, h, flags | ST | B.CAST_F_BULK_STAGING, meta_in, ref)
        U.assert_parity(got, want, f"staged {what} {rows}x{cols}")
        check_stats(got, stats, want, ref, 4, False, f"staged {what} {rows}x{cols} ref={ref is not None}")
        plain, plain_stats = step_with_stats(inp, 2, 4, h, flags | ST | B.CAST_F_PLAIN_ACCESS, meta_in, ref)
        for k in ("w", "m", "v", "w_fwd", "meta"):
            assert np.array_equal(got[k], plain[k]), f"{what}: {k} differs between the access paths"
        assert stats["flips"] == plain_stats["flips"]


def test_plan_step_with_statistics_accumulates_over_matrices():
    """All matrices of a plan in one launch: the accumulator holds the model-wide sums, the reference masks are the
    masks of an earlier step (the initial flip rate i_t of App. C), and the step's own results are unchanged by
    the flag."""
    shapes = [(24, 256), (7, 2080), (3, 1056), (40, 512)]
    plain = DeviceModelState(shapes, 2, 4, seed=5, device=DEV, scale_mode="jitter")
    fused = DeviceModelState(shapes, 2, 4, seed=5, device=DEV, scale_mode="jitter", reference_masks=True)
    h = RunHyper(total_steps=30000)
    for s in (plain, fused):
        s.step(h, RS)                                   # masks of the initial weights
    for mat in fused.mats:
        mat.meta_ref.copy_(mat.meta)                    # M_0
    h.step += 1
    before = {i: workloads.TensorInputs(m.w.cpu(), m.g.cpu(), m.m.cpu(), m.v.cpu(), m.scale.cpu()) for i, m in enumerate(fused.mats)}
    metas = [m.meta.cpu().numpy().view(np.uint32).copy() for m in fused.mats]
    launches = cast.cast_kernel_launch_count()
    fused.step(h, RS | FL | DN | ST)
    plain.step(h, RS | FL | DN)
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == launches + 3       # two steps and one fold
    got = fused.read_stats()
    oh = Hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step, h.total_steps)
    want = dict(flips=0, kept_abs=0.0, total_abs=0.0)
    n = 0
    for i, (a, b) in enumerate(zip(plain.mats, fused.mats)):
        for k in ("w", "m", "v", "w_fwd", "meta"):
            assert torch.equal(getattr(a, k), getattr(b, k)), f"matrix {i} {k}: the statistics flag changed the step's results"
        ref = U.run_oracle(before[i], 2, 4, oh, RS | FL | DN, meta_in=metas[i])
        part = orc.mask_stats(ref["w"], ref["meta"], metas[i], 4, False)
        for k in want:
            want[k] += part[k]
        n += a.rows * a.cols
    assert int(fused.flips.item()) == int(plain.flips.item()) == want["flips"]      # M_ref = M_{t-1} here: i_t = r_t
    assert got.mask_diff == want["flips"]
    assert abs(got.kept_abs_sum - want["kept_abs"]) <= 1e-6 * want["total_abs"] + 1e-9 * n
    assert abs(got.total_abs_sum - want["total_abs"]) <= 1e-6 * want["total_abs"] + 1e-9 * n
    plain.close()
    fused.close()


def test_statistics_flag_needs_a_plan_made_for_it_and_an_accumulator():
    inp = workloads.gen_tensor_inputs(4, 64, seed=3, device="cpu", scale_mode="none")
    st = U.to_device(inp, DEV)
    before = cast.cast_kernel_launch_count()
    rc = cast.cast_adams_step(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, None, 1, 4, 64, 2, 4,
                              1e-4, 0.9, 0.95, 1e-8, 1e-3, 1, 10, RS | ST, None, None)
    assert rc == B.CAST_ERR_PLAN
    t = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, None, 1, 4, 64)
    hy = B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 1e-3, 1, 10, RS | ST)
    assert cast.cast_adams_step_ex(t, 2, 4, hy, None, None) == B.CAST_ERR_PLAN
    stats = torch.zeros(40, dtype=torch.uint8, device=DEV)
    rc, ordinary = B.cast_plan_create([t], 2, 4)
    cast.check(rc)
    assert cast.cast_plan_step_stats(ordinary, hy, None, stats[:32], None) == B.CAST_ERR_PLAN     # not created for statistics
    assert cast.cast_plan_step(ordinary, hy, None, None) == B.CAST_ERR_NULL                        # no accumulator
    cast.check(cast.cast_plan_destroy(ordinary))
    rc, plan = B.cast_plan_create_ex([t], 2, 4, ST)
    cast.check(rc)
    assert cast.cast_plan_step_stats(plan, hy, None, None, None) == B.CAST_ERR_NULL
    assert cast.cast_plan_step_stats(plan, hy, None, stats[4:36], None) == B.CAST_ERR_ALIGN
    cast.check(cast.cast_plan_destroy(plan))
    bad_ref = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, None, 1, 4, 64, None, st.meta.view)
    rc, none = B.cast_plan_create_ex([bad_ref], 2, 4, ST)
    assert rc == B.CAST_ERR_ALIAS and none is None
    assert cast.cast_kernel_launch_count() == before


def test_two_steps_of_one_plan_leave_no_partial_sums_behind():
    """The partial accumulators of the plan are cleared by every step: a second step adds exactly its own sums."""
    shapes = [(16, 512), (5, 96)]
    st = DeviceModelState(shapes, 2, 4, seed=8, device=DEV, scale_mode="jitter", reference_masks=True)
    h = RunHyper(total_steps=30000)
    st.step(h, RS | ST)
    first = st.read_stats()
    st.stats.zero_()
    h.step += 1
    st.step(h, ST)                                    # stored mask, same weights' successors
    second = st.read_stats()
    mag = sum(float(m.w.double().abs().sum().item()) for m in st.mats)
    assert second.total_abs_sum == pytest.approx(mag, rel=1e-12)
    assert first.total_abs_sum != second.total_abs_sum
    st.close()
