"""Full-size workloads in the launch configuration the benchmark times, checked on sampled row blocks
(the oracle recomputes each sampled block from host copies taken before the step) and on properties
that hold at any size."""
import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from paper_2509_25996_b200.runner import DeviceModelState, Hyper as RunHyper
from oracle import adams_oracle as orc
import gpu_util as U
from helpers import within_tol

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def sample_blocks(shapes, n_random, rows_per_block, seed):
    rng = np.random.default_rng(seed)
    picks = [(0, 0), (len(shapes) - 1, shapes[-1][0] - rows_per_block)]      # very first and very last rows
    for _ in range(n_random):
        t = int(rng.integers(0, len(shapes)))
        picks.append((t, int(rng.integers(0, shapes[t][0] - rows_per_block + 1))))
    return picks


def check_sampled(wl_name, N, M, flags, n_random=14, rows_per_block=6, need_gb=0.0):
    import gc
    gc.collect()
    torch.cuda.empty_cache()                                     # blocks cached by earlier tests count as used
    free, _ = torch.cuda.mem_get_info()
    if free < need_gb * 1e9:
        pytest.skip(f"needs {need_gb} GB of device memory, {free / 1e9:.0f} GB free")
    wl = workloads.workload(wl_name)
    state = DeviceModelState(wl.shapes, N, M, seed=0, device=DEV, scale_mode="jitter")
    picks = sample_blocks(wl.shapes, n_random, rows_per_block, seed=1)
    before = []
    for t, r0 in picks:
        s = state.mats[t]
        sl = slice(r0, r0 + rows_per_block)
        before.append(workloads.TensorInputs(s.w[sl].cpu(), s.g[sl].cpu(), s.m[sl].cpu(), s.v[sl].cpu(), s.scale[sl].cpu()))
    h = RunHyper(total_steps=wl.total_steps)
    launches = cast.cast_kernel_launch_count()
    state.step(h, flags)
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == launches + 1
    oh = orc.Hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step, h.total_steps)
    for (t, r0), inp in zip(picks, before):
        s = state.mats[t]
        sl = slice(r0, r0 + rows_per_block)
        got = dict(w=s.w[sl].cpu().numpy(), m=s.m[sl].cpu().numpy(), v=s.v[sl].cpu().numpy(),
                   w_fwd=workloads.bf16_bits(s.w_fwd[sl]), meta=s.meta[sl].cpu().numpy().view(np.uint32))
        U.assert_parity(got, U.run_oracle(inp, N, M, oh, flags), f"{wl_name} tensor {t} rows {r0}+")
    # properties at full size: every group keeps exactly N (Eq. 4), pruned slots are +0, one bit per parameter
    bitmask = bool(flags & B.CAST_F_META_BITMASK)
    for t in (0, len(wl.shapes) // 2, len(wl.shapes) - 1):
        s = state.mats[t]
        nz = (s.w_fwd.view(torch.int16) != 0).view(s.rows, s.cols // M, M).sum(-1)
        assert int(nz.max().item()) <= N and float((nz == N).float().mean().item()) > 0.999
        assert s.meta.numel() * 4 == s.rows * s.cols // 8
        if bitmask:
            pop = sum(((s.meta >> b) & 1).sum(dtype=torch.int64) for b in range(32))
            assert int(pop.item()) == s.rows * s.cols * N // M
    state.close()


def test_llama2_7b_full_set_sampled():
    """LLaMA2-7B linear set (224 matrices, 6,476,005,376 parameters, 104 GB resident), one launch."""
    check_sampled("llama2_7b", 2, 4, B.CAST_F_RESELECT, need_gb=125)


@pytest.mark.parametrize("N,M", [(4, 8), (1, 4)])
def test_llama2_7b_layer_general_nm_sampled(N, M):
    check_sampled("llama2_7b_layer", N, M, B.CAST_F_RESELECT | B.CAST_F_META_BITMASK, n_random=8, need_gb=5)


def test_llama2_7b_full_set_4_8_with_flips_sampled():
    """The full LLaMA2-7B set under 4:8 with flip counting (one launch, bitmask metadata): sampled row blocks
    against the oracle, Eq. 4 on whole matrices, and the flip total is even (groups keep exactly N, so a group
    that changes its kept set changes it in pairs) and equals the mask statistics pass against the old masks."""
    import ctypes
    import gc
    gc.collect()
    torch.cuda.empty_cache()                                     # blocks cached by earlier tests count as used
    free, _ = torch.cuda.mem_get_info()
    if free < 125e9:
        pytest.skip("needs 125 GB of device memory")
    wl = workloads.workload("llama2_7b")
    N, M = 4, 8
    flags = B.CAST_F_RESELECT | B.CAST_F_META_BITMASK
    state = DeviceModelState(wl.shapes, N, M, seed=0, device=DEV, scale_mode="jitter")
    h = RunHyper(total_steps=wl.total_steps)
    state.step(h, flags)                                         # masks of the initial weights
    picks = sample_blocks(wl.shapes, 10, 6, seed=2)
    before, old_meta = [], []
    for t, r0 in picks:
        s = state.mats[t]
        sl = slice(r0, r0 + 6)
        before.append((workloads.TensorInputs(s.w[sl].cpu(), s.g[sl].cpu(), s.m[sl].cpu(), s.v[sl].cpu(), s.scale[sl].cpu()),
                       s.meta[sl].cpu().numpy().view(np.uint32).copy()))
    refs = [m.meta.clone() for m in state.mats[:8]]              # reference masks of the first layer and a bit
    h.step += 1
    state.flips.zero_()
    state.step(h, flags | B.CAST_F_COUNT_FLIPS)
    torch.cuda.synchronize()
    flips = int(state.flips.item())
    assert flips > 0 and flips % 2 == 0
    oh = orc.Hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step, h.total_steps)
    sampled_flips = 0
    for (t, r0), (inp, meta_in) in zip(picks, before):
        s = state.mats[t]
        sl = slice(r0, r0 + 6)
        got = dict(w=s.w[sl].cpu().numpy(), m=s.m[sl].cpu().numpy(), v=s.v[sl].cpu().numpy(),
                   w_fwd=workloads.bf16_bits(s.w_fwd[sl]), meta=s.meta[sl].cpu().numpy().view(np.uint32))
        ref = U.run_oracle(inp, N, M, oh, flags | B.CAST_F_COUNT_FLIPS, meta_in=meta_in)
        U.assert_parity(got, ref, f"4:8 tensor {t} rows {r0}+")
        sampled_flips += ref["flips"]
    assert sampled_flips <= flips
    # the flips of the first matrices, counted a second way by the statistics pass
    stats = torch.zeros(ctypes.sizeof(B.cast_mask_stats_t), dtype=torch.uint8, device=DEV)
    part = 0
    for mat, ref_meta in zip(state.mats[:8], refs):
        cast.check(cast.cast_mask_stats(mat.w, mat.meta, ref_meta, mat.rows, mat.cols, M, B.CAST_F_META_BITMASK, stats, None))
        pop = sum((((mat.meta ^ ref_meta) >> b) & 1).sum(dtype=torch.int64) for b in range(32))
        part += int(pop.item())
    torch.cuda.synchronize()
    assert B.cast_mask_stats_t.from_buffer_copy(stats.cpu().numpy().tobytes()).mask_diff == part
    for t in (0, len(wl.shapes) - 1):
        s = state.mats[t]
        pop = sum(((s.meta >> b) & 1).sum(dtype=torch.int64) for b in range(32))
        assert int(pop.item()) == s.rows * s.cols * N // M
    state.close()


def test_llama2_13b_layer_sampled():
    check_sampled("llama2_13b_layer", 2, 4, B.CAST_F_RESELECT, n_random=8, need_gb=8)


def test_llama2_13b_streamed_full_sampled():
    """LLaMA2-13B layer shapes, 40 layers in per-layer calls on 2 streams over 10 resident layer slots (51 GB): every
    slot takes 4 steps per pass; sampled row blocks of slots 0 and 9 against 4 chained oracle steps."""
    import gc
    from paper_2509_25996_b200.runner import StreamedModelState
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 60e9:
        pytest.skip("needs 60 GB of device memory")
    wl = workloads.workload("llama2_13b")
    layer = wl.shapes[:wl.layer_matrices]
    st = StreamedModelState(layer, len(wl.shapes) // wl.layer_matrices, wl.resident_layers, 2, 2, 4, seed=0, device=DEV,
                            scale_mode="jitter")
    rng = np.random.default_rng(3)
    picks = [(slot, t, int(rng.integers(0, layer[t][0] - 4))) for slot in (0, 9) for t in (0, 4, 6)]
    before = []
    for slot, t, r0 in picks:
        m = st.slots[slot].mats[t]
        sl = slice(r0, r0 + 4)
        before.append(workloads.TensorInputs(m.w[sl].cpu(), m.g[sl].cpu(), m.m[sl].cpu(), m.v[sl].cpu(), m.scale[sl].cpu()))
    h = RunHyper(total_steps=wl.total_steps)
    launches = cast.cast_kernel_launch_count()
    st.step(h, B.CAST_F_RESELECT)
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == launches + 40
    oh = orc.Hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step, h.total_steps)
    for (slot, t, r0), inp in zip(picks, before):
        cur = inp
        for _ in range(4):
            ref = U.run_oracle(cur, 2, 4, oh, B.CAST_F_RESELECT)
            cur = workloads.TensorInputs(torch.from_numpy(ref["w"]), inp.g, torch.from_numpy(ref["m"]), torch.from_numpy(ref["v"]), inp.scale)
        m = st.slots[slot].mats[t]
        sl = slice(r0, r0 + 4)
        got = dict(w=m.w[sl].cpu().numpy(), m=m.m[sl].cpu().numpy(), v=m.v[sl].cpu().numpy())
        # four chained steps: the fp32 state of one step feeds the next, so the bound grows with the step count
        for k in ("w", "m", "v"):
            ok, worst = within_tol(got[k], ref[k], rel=4e-6, floor=4e-9)
            assert ok, f"slot {slot} matrix {t} rows {r0}+ {k}: {worst:.3g}"
    st.close()
