"""cast_prune_fold (final pruning with the scale folded in, Alg. 2's last loop) against the CPU oracle: values and
metadata bit-exact (the product a*w is one fp32 rounding and one bf16 rounding on both sides... the oracle forms
the product in fp64, so a value may differ by one bf16 ulp where the fp32 product lands on a rounding boundary)."""
import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle import adams_oracle as orc
from helpers import bf16_ulp_distance
import gpu_util as U

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RS, BM, C = B.CAST_F_RESELECT, B.CAST_F_META_BITMASK, B.CAST_F_EMIT_COMPRESSED


def oracle_flags(flags):
    return (orc.F_RESELECT if flags & RS else 0) | (orc.F_META_BITMASK if flags & BM else 0) | (orc.F_EMIT_COMPRESSED if flags & C else 0)


def run_gpu(w, scale, N, M, flags, meta_in=None):
    rows, cols = w.shape
    n_out = rows * cols * N // M if flags & C else rows * cols
    d_w = U.Guarded(rows * cols, torch.float32, DEV, w.to(DEV))
    out = U.Guarded(n_out, torch.bfloat16, DEV)
    meta = U.Guarded(rows * cols // 32, torch.int32, DEV)
    if meta_in is not None:
        meta.view.copy_(torch.from_numpy(meta_in.view(np.int32).reshape(-1).copy()))
    d_scale = None if scale is None else scale.to(DEV).contiguous()
    before = cast.cast_kernel_launch_count()
    cast.check(cast.cast_prune_fold(d_w.view, d_scale, 1 if scale is None else scale.shape[1], meta.view, out.view,
                                    rows, cols, N, M, flags, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + 1
    assert d_w.intact() and out.intact() and meta.intact()
    assert torch.equal(d_w.view.cpu(), w.reshape(-1))                      # the weights are only read
    return workloads.bf16_bits(out.view).reshape(rows, -1), meta.view.cpu().numpy().view(np.uint32).reshape(rows, cols // 32)


def check(w, scale, N, M, flags, meta_in=None, label=""):
    got_out, got_meta = run_gpu(w, scale, N, M, flags, meta_in)
    ref = orc.prune_fold(w.numpy(), None if scale is None else scale.numpy(), N, M, oracle_flags(flags), meta_in)
    assert np.array_equal(got_meta, ref["meta"]), f"{label}: metadata differs"
    d = bf16_ulp_distance(got_out, ref["out"])
    assert d.max(initial=0) <= 1 and np.mean(d != 0) < 1e-3, f"{label}: values differ by {d.max()} ulp"
    assert np.array_equal(got_out == 0, ref["out"] == 0) or np.all((got_out & 0x7FFF)[(got_out == 0) != (ref["out"] == 0)] <= 1)


@pytest.mark.parametrize("N,M", [(2, 4), (1, 4), (3, 4), (1, 2), (4, 8), (3, 8), (8, 8), (5, 16), (8, 32)])
@pytest.mark.parametrize("compressed", [False, True])
def test_prune_fold_every_nm(N, M, compressed):
    if compressed and M > 8:
        pytest.skip("the compressed form needs M <= 8")
    rows, cols = 7, 2080
    inp = workloads.gen_tensor_inputs(rows, cols, seed=300 + M, tensor_index=N, scale_mode="jitter")
    scale = inp.scale if (cols // 2) % max(M, 8) == 0 else None
    extra = C if compressed else 0
    for enc in ([0, BM] if (N, M) == (2, 4) else [BM]):
        check(inp.w, scale, N, M, RS | enc | extra, label=f"{N}:{M} enc {enc} compressed {compressed}")
        # a stored mask (of other weights) is used as it is
        stored = orc.prune_fold(workloads.gen_tensor_inputs(rows, cols, seed=400 + M).w.numpy(), None, N, M,
                                orc.F_RESELECT | (orc.F_META_BITMASK if enc else 0))["meta"]
        check(inp.w, scale, N, M, enc | extra, meta_in=stored, label=f"{N}:{M} stored mask")


def test_prune_fold_adversarial_values_and_exact_scale():
    rows, cols = 12, 384
    rng = np.random.default_rng(5)
    w = torch.from_numpy(rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32))
    g = w.view(-1, 4)
    g[0::9, 1] = g[0::9, 0]; g[1::9, 3] = -g[1::9, 0]; g[2::9, :] = 0.0; g[3::9, 0] = -0.0
    g[4::9, :] = 0.125; g[5::9, 0] = 1e-41; g[6::9, 0] = 3e4; g[6::9, 1] = 1e-30
    scale = torch.from_numpy(np.ldexp(1.0, rng.integers(-3, 4, size=(rows, 2))).astype(np.float32))   # exact products
    for flags in (RS, RS | BM, RS | C, RS | BM | C):
        got_out, got_meta = run_gpu(w, scale, 2, 4, flags)
        ref = orc.prune_fold(w.numpy(), scale.numpy(), 2, 4, oracle_flags(flags))
        assert np.array_equal(got_meta, ref["meta"]) and np.array_equal(got_out, ref["out"])           # bit for bit


@pytest.mark.parametrize("N,M,enc,compressed", [(2, 4, 0, False), (2, 4, 0, True), (4, 8, BM, True), (8, 16, BM, False)])
def test_plan_prune_fold_one_launch(N, M, enc, compressed):
    """Every matrix of a plan in one grid: ragged tiles, one-unit matrices, with and without a scale."""
    shapes = [(1, 32), (3, 96), (64, 1056), (7, 2080), (1, 32), (33, 2048)]
    extra = C if compressed else 0
    ins = [workloads.gen_tensor_inputs(r, c, seed=310, tensor_index=i, scale_mode="jitter" if (c // 2) % max(M, 8) == 0 else "none")
           for i, (r, c) in enumerate(shapes)]
    states = [U.to_device(inp, DEV) for inp in ins]
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale,
                             1 if s.scale is None else s.scale.shape[1], s.rows, s.cols) for s in states]
    rc, plan = cast.cast_plan_create(tensors, N, M)
    cast.check(rc)
    outs = [U.Guarded(r * c * N // M if compressed else r * c, torch.bfloat16, DEV) for r, c in shapes]
    before = cast.cast_kernel_launch_count()
    cast.check(cast.cast_plan_prune_fold(plan, [o.view for o in outs], RS | enc | extra, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + 1
    for i, (s, inp, o) in enumerate(zip(states, ins, outs)):
        assert s.all_intact() and o.intact()
        ref = orc.prune_fold(inp.w.numpy(), None if inp.scale is None else inp.scale.numpy(), N, M, oracle_flags(RS | enc | extra))
        assert np.array_equal(s.meta.view.cpu().numpy().view(np.uint32).reshape(ref["meta"].shape), ref["meta"]), f"tensor {i}"
        d = bf16_ulp_distance(workloads.bf16_bits(o.view).reshape(ref["out"].shape), ref["out"])
        assert d.max(initial=0) <= 1, f"tensor {i}"
        assert torch.equal(s.w.view.cpu(), inp.w.reshape(-1))                 # state untouched
    assert cast.cast_plan_prune_fold(plan, None, RS | enc, None) == B.CAST_ERR_NULL
    assert cast.cast_plan_prune_fold(None, [o.view for o in outs], RS | enc, None) == B.CAST_ERR_PLAN
    assert cast.cast_plan_prune_fold(plan, [s.w.view for s in states], RS | enc, None) == B.CAST_ERR_ALIAS
    cast.check(cast.cast_plan_destroy(plan))


def test_prune_fold_rejections():
    w = torch.zeros(4 * 64, device=DEV)
    meta = torch.zeros(4 * 2, dtype=torch.int32, device=DEV)
    out = torch.zeros(4 * 64, dtype=torch.bfloat16, device=DEV)
    before = cast.cast_kernel_launch_count()
    assert cast.cast_prune_fold(None, None, 1, meta, out, 4, 64, 2, 4, RS) == B.CAST_ERR_NULL
    assert cast.cast_prune_fold(w, None, 1, meta, out, 4, 64, 4, 8, RS) == B.CAST_ERR_NM                 # index form is 2:4 only
    assert cast.cast_prune_fold(w, None, 1, meta, out, 4, 64, 8, 16, RS | BM | C) == B.CAST_ERR_NM
    assert cast.cast_prune_fold(w, None, 1, meta, out, 4, 64, 2, 4, RS | B.CAST_F_COUNT_FLIPS) == B.CAST_ERR_HYPER
    assert cast.cast_prune_fold(w, None, 1, meta, out, 4, 48, 2, 4, RS) == B.CAST_ERR_SHAPE
    assert cast.cast_prune_fold(w, None, 1, meta, w, 4, 64, 2, 4, RS) == B.CAST_ERR_ALIAS
    assert cast.cast_prune_fold(torch.zeros(4 * 64), None, 1, meta, out, 4, 64, 2, 4, RS) == B.CAST_ERR_MEMORY
    assert cast.cast_kernel_launch_count() == before
