"""The gradient taken through the weight scaling of Eq. 12 (CAST_F_GRAD_OF_SCALED), the fused scale gradient and
the Adam step of the scale matrix, against the CPU oracle.

Tolerances: w, m, v, w_fwd, metadata as everywhere else.  The scale gradient is an fp32 sum of cols/n products
formed in an order that varies between runs (eight fused multiply-adds per thread, a warp scan, atomics), the
oracle's is an fp64 sum: |cuda - oracle| <= 2e-6 * sum |g w| over the segment.  The scale's Adam step runs in
fp64 on both sides: 1e-6 relative covers the fp32 rounding of the stored results."""
import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle import adams_oracle as orc
from oracle.adams_oracle import Hyper
import gpu_util as U

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RS, BM, GS = B.CAST_F_RESELECT, B.CAST_F_META_BITMASK, B.CAST_F_GRAD_OF_SCALED


def hyper_struct(h: Hyper, flags):
    lr, b1, b2, eps, lam = h.as_f32()
    return B.make_hyper(lr, b1, b2, eps, lam, h.step, h.total_steps, flags)


def scaled_inputs(rows, cols, n_seg, seed):
    inp = workloads.gen_tensor_inputs(rows, cols, seed=seed, scale_mode="jitter")
    gen = torch.Generator().manual_seed(seed + 1000)
    inp.scale = 0.5 + torch.rand((rows, n_seg), generator=gen)
    return inp


def assert_scale_grad(got, inp, ref, n_seg, label, start=None):
    rows, cols = inp.w.shape
    g32 = inp.g.to(torch.float64).numpy()
    bound = 2e-6 * np.abs(g32 * inp.w.to(torch.float64).numpy()).reshape(rows, n_seg, cols // n_seg).sum(-1) + 1e-30
    want = ref if start is None else ref + start
    err = np.abs(got.astype(np.float64) - want)
    assert np.all(err <= bound + 1e-6 * np.abs(want) * (start is not None)), f"{label}: worst {np.max(err / bound):.3g} x the bound"


@pytest.mark.parametrize("rows,cols,n_seg", [(1, 32, 1), (3, 96, 2), (5, 2080, 2), (7, 1024, 4), (4, 2304, 48), (9, 11008, 2)])
@pytest.mark.parametrize("N,M,extra", [(2, 4, 0), (4, 8, BM), (8, 16, BM)])
def test_step_with_gradient_of_scaled_weight(rows, cols, n_seg, N, M, extra):
    """Segments of 1 to 688 units: shorter than a warp, straddling warps and tiles, several per warp."""
    if (cols // n_seg) % max(M, 8) != 0:
        pytest.skip("segment not a multiple of the group")
    inp = scaled_inputs(rows, cols, n_seg, seed=200 + n_seg)
    h = Hyper()
    flags = RS | extra | GS
    st = U.to_device(inp, DEV)
    sg = torch.zeros((rows, n_seg), dtype=torch.float32, device=DEV)
    t = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, st.scale, n_seg, rows, cols, sg)
    cast.check(cast.cast_adams_step_ex(t, N, M, hyper_struct(h, flags), None, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert st.all_intact()
    ref = U.run_oracle(inp, N, M, h, flags)
    U.assert_parity(U.device_outputs(st), ref, f"grad of scaled {N}:{M} {rows}x{cols}/{n_seg}")
    assert_scale_grad(sg.cpu().numpy(), inp, ref["scale_grad"], n_seg, f"scale grad {rows}x{cols}/{n_seg}")


@pytest.mark.parametrize("flags", [B.CAST_F_EMIT_DENSE | GS, RS | B.CAST_F_COUNT_FLIPS | B.CAST_F_EMIT_DENSE | GS])
def test_training_steps_with_a_learned_scale(flags):
    """The two steps of training with a learned scale (Alg. 2 with Eq. 12): the common one (stored mask, dense
    forward weight, gradient through the scaling) and the refresh one (mask reselected, flips counted)."""
    rows, cols, n_seg = 9, 2080, 2
    inp = scaled_inputs(rows, cols, n_seg, seed=230)
    h = Hyper()
    stored = U.run_oracle(scaled_inputs(rows, cols, n_seg, seed=231), 2, 4, h, RS)["meta"]
    st = U.to_device(inp, DEV, stored)
    sg = torch.zeros((rows, n_seg), dtype=torch.float32, device=DEV)
    flips = torch.zeros(1, dtype=torch.int64, device=DEV)
    t = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, st.scale, n_seg, rows, cols, sg)
    cast.check(cast.cast_adams_step_ex(t, 2, 4, hyper_struct(h, flags), flips, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert st.all_intact()
    ref = U.run_oracle(inp, 2, 4, h, flags, meta_in=stored)
    got = U.device_outputs(st)
    U.assert_parity(got, ref, f"learned scale, flags {flags}")
    assert_scale_grad(sg.cpu().numpy(), inp, ref["scale_grad"], n_seg, "scale grad")
    if flags & B.CAST_F_COUNT_FLIPS:
        assert int(flips.item()) == ref["flips"] > 0
    else:
        assert np.array_equal(got["meta"], stored)


def test_scale_gradient_is_added_and_optional_and_plain_step_is_unchanged():
    rows, cols, n_seg = 6, 1056, 2
    inp = scaled_inputs(rows, cols, n_seg, seed=210)
    h = Hyper()
    ref = U.run_oracle(inp, 2, 4, h, RS | GS)
    # added to what the buffer holds
    st = U.to_device(inp, DEV)
    start = torch.full((rows, n_seg), 0.25, dtype=torch.float32, device=DEV)
    sg = start.clone()
    t = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, st.scale, n_seg, rows, cols, sg)
    cast.check(cast.cast_adams_step_ex(t, 2, 4, hyper_struct(h, RS | GS), None, None))
    torch.cuda.synchronize()
    assert_scale_grad(sg.cpu().numpy(), inp, ref["scale_grad"], n_seg, "accumulated", start=0.25)
    # without a buffer the chain rule to W is still applied
    st2 = U.to_device(inp, DEV)
    t2 = B.make_tensor(st2.w.view, st2.m.view, st2.v.view, st2.g.view, st2.w_fwd.view, st2.meta.view, st2.scale, n_seg, rows, cols)
    cast.check(cast.cast_adams_step_ex(t2, 2, 4, hyper_struct(h, RS | GS), None, None))
    torch.cuda.synchronize()
    U.assert_parity(U.device_outputs(st2), ref, "no scale-grad buffer")
    # the structure form without the flag is the plain entry point, bit for bit
    a = U.run_cuda_single(inp, 2, 4, h, RS)
    st3 = U.to_device(inp, DEV)
    t3 = B.make_tensor(st3.w.view, st3.m.view, st3.v.view, st3.g.view, st3.w_fwd.view, st3.meta.view, st3.scale, n_seg, rows, cols)
    cast.check(cast.cast_adams_step_ex(t3, 2, 4, hyper_struct(h, RS), None, None))
    torch.cuda.synchronize()
    b = U.device_outputs(st3)
    for k in ("w", "m", "v", "w_fwd", "meta"):
        assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8))
    # a scale gradient needs a scale
    before = cast.cast_kernel_launch_count()
    t4 = B.make_tensor(st3.w.view, st3.m.view, st3.v.view, st3.g.view, st3.w_fwd.view, st3.meta.view, None, 1, rows, cols, sg)
    assert cast.cast_adams_step_ex(t4, 2, 4, hyper_struct(h, RS | GS), None, None) == B.CAST_ERR_NULL
    assert cast.cast_adams_step_ex(None, 2, 4, hyper_struct(h, RS), None, None) == B.CAST_ERR_NULL
    assert cast.cast_kernel_launch_count() == before


def test_plan_with_scale_gradients_then_scale_adam():
    """One training iteration of weights and scales: a plan step with the chain rule and fused scale gradients,
    then the Adam step of every scale matrix, against the oracle's two routines."""
    shapes = [(3, 96), (64, 1056), (7, 2080), (33, 2048)]
    h = Hyper()
    ins = [scaled_inputs(r, c, 2, seed=220 + i) for i, (r, c) in enumerate(shapes)]
    states = [U.to_device(inp, DEV) for inp in ins]
    grads = [torch.zeros((r, 2), dtype=torch.float32, device=DEV) for r, _ in shapes]
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale, 2, s.rows, s.cols, gr)
               for s, gr in zip(states, grads)]
    rc, plan = cast.cast_plan_create(tensors, 2, 4)
    cast.check(rc)
    stream = torch.cuda.current_stream()
    cast.check(cast.cast_plan_step(plan, hyper_struct(h, RS | GS), None, stream))
    torch.cuda.synchronize()
    lr_a = float(np.float32(1e-3))
    for i, (s, inp, gr) in enumerate(zip(states, ins, grads)):
        ref = U.run_oracle(inp, 2, 4, h, RS | GS)
        U.assert_parity(U.device_outputs(s), ref, f"plan tensor {i}")
        got_grad = gr.cpu().numpy()
        assert_scale_grad(got_grad, inp, ref["scale_grad"], 2, f"plan scale grad {i}")
        # Adam on the scale from the gradient the CUDA path produced (so both sides start from the same numbers)
        n = s.rows * 2
        m_a = torch.zeros(n, dtype=torch.float32, device=DEV)
        v_a = torch.zeros(n, dtype=torch.float32, device=DEV)
        a0 = s.scale.cpu().numpy().reshape(-1).copy()
        for t in (1, 2):
            gr.copy_(torch.from_numpy(got_grad * t))
            cast.check(cast.cast_scale_adam_step(s.scale, m_a, v_a, gr, n, lr_a, 0.9, 0.95, 1e-8, t, True, stream))
        torch.cuda.synchronize()
        assert float(gr.abs().max().item()) == 0.0                                   # cleared for the next iteration
        th, mm, vv = a0, np.zeros(n, np.float32), np.zeros(n, np.float32)
        for t in (1, 2):
            th, mm, vv = orc.plain_adam(th, mm, vv, (got_grad * t).reshape(-1), lr_a, 0.9, 0.95, 1e-8, t)
        for got, want in ((s.scale, th), (m_a, mm), (v_a, vv)):
            assert np.allclose(got.cpu().numpy().reshape(-1), want, rtol=1e-6, atol=1e-30)
    cast.check(cast.cast_plan_destroy(plan))
    assert all(s.all_intact() for s in states)


def test_plan_scale_adam_one_launch():
    """The Adam step of every scale matrix of a plan in one grid (scale matrices of 2 to 600 entries)."""
    shapes = [(1, 64), (3, 96), (64, 1056), (300, 64), (33, 2048)]
    ins = [scaled_inputs(r, c, 2, seed=240 + i) for i, (r, c) in enumerate(shapes)]
    states = [U.to_device(inp, DEV) for inp in ins]
    rng = np.random.default_rng(7)
    grads_h = [rng.normal(0, 1e-2, size=(r, 2)).astype(np.float32) for r, _ in shapes]
    grads = [torch.from_numpy(g.copy()).to(DEV) for g in grads_h]
    m_as = [torch.zeros(r * 2, device=DEV) for r, _ in shapes]
    v_as = [torch.zeros(r * 2, device=DEV) for r, _ in shapes]
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale, 2, s.rows, s.cols, gr)
               for s, gr in zip(states, grads)]
    rc, plan = cast.cast_plan_create(tensors, 2, 4)
    cast.check(rc)
    lr_a = float(np.float32(1e-3))
    before = cast.cast_kernel_launch_count()
    cast.check(cast.cast_plan_scale_adam_step(plan, m_as, v_as, lr_a, 0.9, 0.95, 1e-8, 3, True, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + 1
    for s, inp, gh, gr, ma, va in zip(states, ins, grads_h, grads, m_as, v_as):
        n = s.rows * 2
        th, mm, vv = orc.plain_adam(inp.scale.numpy().reshape(-1), np.zeros(n, np.float32), np.zeros(n, np.float32),
                                    gh.reshape(-1), lr_a, 0.9, 0.95, 1e-8, 3)
        for got, want in ((s.scale, th), (ma, mm), (va, vv)):
            assert np.allclose(got.cpu().numpy().reshape(-1), want, rtol=1e-6, atol=1e-30)
        assert float(gr.abs().max().item()) == 0.0
        assert s.all_intact()
    assert cast.cast_plan_scale_adam_step(plan, None, v_as, lr_a, 0.9, 0.95, 1e-8, 3) == B.CAST_ERR_NULL
    assert cast.cast_plan_scale_adam_step(None, m_as, v_as, lr_a, 0.9, 0.95, 1e-8, 3) == B.CAST_ERR_PLAN
    assert cast.cast_plan_scale_adam_step(plan, m_as, v_as, lr_a, 0.9, 0.95, 1e-8, 0) == B.CAST_ERR_HYPER
    cast.check(cast.cast_plan_destroy(plan))
    # a plan whose matrices carry no scale gradient cannot train the scale
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale, 2, s.rows, s.cols) for s in states]
    rc, plan = cast.cast_plan_create(tensors, 2, 4)
    cast.check(rc)
    assert cast.cast_plan_scale_adam_step(plan, m_as, v_as, lr_a, 0.9, 0.95, 1e-8, 3) == B.CAST_ERR_NULL
    cast.check(cast.cast_plan_destroy(plan))


def test_scale_adam_rejections():
    x = torch.zeros(64, dtype=torch.float32, device=DEV)
    y, z, g = x.clone(), x.clone(), x.clone()
    before = cast.cast_kernel_launch_count()
    assert cast.cast_scale_adam_step(x, y, z, None, 64, 1e-3, 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_NULL
    assert cast.cast_scale_adam_step(x, y, z, g, 0, 1e-3, 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_SHAPE
    assert cast.cast_scale_adam_step(x, y, z, g, 64, 1e-3, 1.0, 0.95, 1e-8, 1) == B.CAST_ERR_HYPER
    assert cast.cast_scale_adam_step(x, y, z, g, 64, 1e-3, 0.9, 0.95, 0.0, 1) == B.CAST_ERR_HYPER
    assert cast.cast_scale_adam_step(x, y, z, g, 64, 1e-3, 0.9, 0.95, 1e-8, 0) == B.CAST_ERR_HYPER
    assert cast.cast_scale_adam_step(x, x, z, g, 64, 1e-3, 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_ALIAS
    assert cast.cast_scale_adam_step(x, y, z, torch.zeros(64), 64, 1e-3, 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_MEMORY
    assert cast.cast_kernel_launch_count() == before


@pytest.mark.parametrize("N,M,extra", [(2, 4, 0), (2, 4, B.CAST_F_EMIT_DENSE), (4, 8, BM), (8, 16, BM)])
def test_chain_rule_with_the_scale_of_the_forward_pass(N, M, extra):
    """A trained scale: the forward pass that produced g was emitted with A_old (`scale_chain`), this step emits with
    the updated A_new (`scale`).  The chain rule must use A_old, the emission A_new, exactly as the oracle does."""
    rows, cols, n_seg = 5, 2080 if M <= 8 else 2048, 2
    inp = scaled_inputs(rows, cols, n_seg, seed=260)
    gen = torch.Generator().manual_seed(261)
    a_old = (inp.scale * (1.0 + 0.05 * torch.rand((rows, n_seg), generator=gen))).contiguous()
    h = Hyper()
    flags = RS | extra | GS
    st = U.to_device(inp, DEV)
    sg = torch.zeros((rows, n_seg), dtype=torch.float32, device=DEV)
    chain = a_old.to(DEV)
    t = B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, st.scale, n_seg, rows, cols, sg, None, chain)
    cast.check(cast.cast_adams_step_ex(t, N, M, hyper_struct(h, flags), None, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert st.all_intact()
    ref = U.run_oracle(inp, N, M, h, flags, scale_chain=a_old.numpy())
    U.assert_parity(U.device_outputs(st), ref, f"two scales {N}:{M}")
    assert_scale_grad(sg.cpu().numpy(), inp, ref["scale_grad"], n_seg, "scale grad with two scales")
    same = U.run_oracle(inp, N, M, h, flags)                        # and it does differ from the one-scale result
    assert not np.array_equal(same["m"], ref["m"])


def test_plan_scale_adam_keeps_the_previous_scale_for_the_next_chain_rule():
    """Two iterations of weights and scales through a plan with `scale_chain` buffers: the scale Adam step stores each
    scale's value before its update, and the next AdamS step's chain rule uses that stored value while its emission
    uses the updated scale -- checked against the oracle fed the two scales the same way."""
    from paper_2509_25996_b200.runner import DeviceModelState, Hyper as RunHyper
    shapes = [(6, 1056), (9, 2048)]
    st = DeviceModelState(shapes, 2, 4, seed=11, device=DEV, scale_mode="jitter", learned_scale=True)
    h = RunHyper(total_steps=30000)
    flags = RS | GS | B.CAST_F_EMIT_DENSE | B.CAST_F_PLAIN_ACCESS
    st.step(h, flags)                                               # iteration 1: chain = scale (initially equal)
    a_before = [m.scale.clone() for m in st.mats]
    st.scale_step(1e-2, h)                                          # A_1 -> A_2; chain buffers now hold A_1
    torch.cuda.synchronize()
    for m, a0 in zip(st.mats, a_before):
        assert torch.equal(m.scale_chain, a0) and not torch.equal(m.scale, a0)
    h.step += 1
    st.fresh_gradients(h.step)
    snaps = [workloads.TensorInputs(m.w.cpu(), m.g.cpu(), m.m.cpu(), m.v.cpu(), m.scale.cpu()) for m in st.mats]
    chains = [m.scale_chain.cpu().numpy() for m in st.mats]
    st.step(h, flags)                                               # iteration 2: chain rule with A_1, emission with A_2
    torch.cuda.synchronize()
    oh = orc.Hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step, h.total_steps)
    for i, (m, inp, ch) in enumerate(zip(st.mats, snaps, chains)):
        got = dict(w=m.w.cpu().numpy(), m=m.m.cpu().numpy(), v=m.v.cpu().numpy(), w_fwd=workloads.bf16_bits(m.w_fwd),
                   meta=m.meta.cpu().numpy().view(np.uint32))
        U.assert_parity(got, U.run_oracle(inp, 2, 4, oh, flags & ~B.CAST_F_PLAIN_ACCESS, scale_chain=ch), f"iteration 2 matrix {i}")
    st.close()
