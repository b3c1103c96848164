"""Multi-tensor plan (one launch over all matrices) and host-resident state, against the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle.adams_oracle import Hyper
import gpu_util as U
from helpers import within_tol

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RS, BM = B.CAST_F_RESELECT, B.CAST_F_META_BITMASK


def pinned(t: torch.Tensor) -> torch.Tensor:
    return t.contiguous().pin_memory()


def run_plan(inputs_list, N, M, hyper: Hyper, flags, metas=None, launches=1):
    states = [U.to_device(inp, DEV, None if metas is None else metas[i]) for i, inp in enumerate(inputs_list)]
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale,
                             1 if s.scale is None else s.scale.shape[1], s.rows, s.cols) for s in states]
    rc, plan = cast.cast_plan_create(tensors, N, M)
    cast.check(rc)
    flips = torch.zeros(1, dtype=torch.int64, device=DEV) if flags & B.CAST_F_COUNT_FLIPS else None
    lr, b1, b2, eps, lam = hyper.as_f32()
    before = cast.cast_kernel_launch_count()
    cast.check(cast.cast_plan_step(plan, B.make_hyper(lr, b1, b2, eps, lam, hyper.step, hyper.total_steps, flags),
                                   flips, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + launches   # one grid covers up to 320 matrices
    cast.check(cast.cast_plan_destroy(plan))
    assert all(s.all_intact() for s in states)
    return [U.device_outputs(s) for s in states], (None if flips is None else int(flips.item()))


def test_plan_mixed_shapes_ragged_tiles():
    """Matrices of 0.03 to 66 tiles, most with a ragged last tile, some without a scale tensor."""
    shapes = [(1, 32), (3, 96), (64, 1056), (7, 2080), (1, 2048), (33, 2048), (5, 416), (2, 64), (40, 800)]
    ins = [workloads.gen_tensor_inputs(r, c, seed=20, tensor_index=i, device="cpu",
                                       scale_mode=("none" if i % 3 == 0 else "jitter")) for i, (r, c) in enumerate(shapes)]
    h = Hyper()
    fl = RS | B.CAST_F_COUNT_FLIPS
    prev = [U.run_oracle(workloads.gen_tensor_inputs(r, c, seed=21, tensor_index=i), 2, 4, h, RS)["meta"]
            for i, (r, c) in enumerate(shapes)]
    got, flips = run_plan(ins, 2, 4, h, fl, prev)
    total = 0
    for i, inp in enumerate(ins):
        ref = U.run_oracle(inp, 2, 4, h, fl, meta_in=prev[i])
        U.assert_parity(got[i], ref, f"tensor {i} {shapes[i]}")
        total += ref["flips"]
    assert flips == total


def test_plan_many_small_matrices_around_a_large_one():
    """More than 256 tiles in total, so one entry of the tile-to-matrix hint table covers several tiles,
    and dozens of one-tile matrices share an entry: the forward walk from the hint takes many steps."""
    shapes = [(1, 32)] * 37 + [(4096, 2304)] + [(1, 64)] * 5 + [(2, 1024)] + [(1, 32)] * 3
    ins = [workloads.gen_tensor_inputs(r, c, seed=24, tensor_index=i, scale_mode=("none" if c < 64 else "jitter"))
           for i, (r, c) in enumerate(shapes)]
    got, _ = run_plan(ins, 2, 4, Hyper(), RS)
    for i, inp in enumerate(ins):
        U.assert_parity(got[i], U.run_oracle(inp, 2, 4, Hyper(), RS), f"tensor {i} {shapes[i]}")


def test_plan_more_matrices_than_one_launch_holds():
    """A launch carries the descriptors of at most 320 matrices: 400 small matrices take two launches."""
    shapes = [(1 + i % 3, 32 * (1 + i % 5)) for i in range(400)]
    ins = [workloads.gen_tensor_inputs(r, c, seed=25, tensor_index=i, scale_mode="none") for i, (r, c) in enumerate(shapes)]
    fl = RS | B.CAST_F_COUNT_FLIPS
    got, flips = run_plan(ins, 2, 4, Hyper(), fl, launches=2)
    total = 0
    for i, inp in enumerate(ins):
        ref = U.run_oracle(inp, 2, 4, Hyper(), fl)
        U.assert_parity(got[i], ref, f"tensor {i} {shapes[i]}")
        total += ref["flips"]
    assert flips == total


@pytest.mark.parametrize("N,M", [(4, 8), (1, 4), (8, 16)])
def test_plan_general_nm(N, M):
    shapes = [(16, 512), (9, 1184), (3, 4096)]
    ins = [workloads.gen_tensor_inputs(r, c, seed=22, tensor_index=i, scale_mode="jitter") for i, (r, c) in enumerate(shapes)]
    got, _ = run_plan(ins, N, M, Hyper(total_steps=7500), RS | BM)
    for i, inp in enumerate(ins):
        U.assert_parity(got[i], U.run_oracle(inp, N, M, Hyper(total_steps=7500), RS | BM), f"{N}:{M} tensor {i}")


def test_plan_decoder_d768_12_layers_full():
    """All 72 linear weights of the 12-layer d=768 decoder (84,934,656 parameters), one launch, compared in full."""
    wl = workloads.workload("decoder_d768_12l")
    h = Hyper(total_steps=wl.total_steps)
    ins = []
    for i, (r, c) in enumerate(wl.shapes):
        t = workloads.gen_tensor_inputs(r, c, seed=0, tensor_index=i, device=DEV, scale_mode="jitter")
        ins.append(workloads.TensorInputs(t.w.cpu(), t.g.cpu(), t.m.cpu(), t.v.cpu(), t.scale.cpu()))
    got, _ = run_plan(ins, 2, 4, h, RS)
    ties = 0
    for i, inp in enumerate(ins):
        U.assert_parity(got[i], U.run_oracle(inp, 2, 4, h, RS), f"tensor {i} {wl.shapes[i]}")
        ties += U.near_tie_groups(inp.w.numpy(), 2, 4)
    print(f"near-tie groups: {ties} of {wl.n_params // 4}; mask mismatches: 0")


@pytest.mark.parametrize("case", range(16))
def test_random_plans(case):
    """Random lists of matrices, N:M, flags, scale segments and scale-gradient buffers through the multi-tensor path."""
    rng = np.random.default_rng(3000 + case)
    M = int(rng.choice([2, 4, 8, 16, 32]))
    N = int(rng.integers(1, M + 1))
    if case % 3 == 0:
        N, M = 2, 4
    flags = RS if rng.random() < 0.7 else 0
    if (N, M) != (2, 4) or rng.random() < 0.5:
        flags |= BM
    for bit, p in ((B.CAST_F_COUNT_FLIPS, 0.5), (B.CAST_F_V_KEPT_FROM_G, 0.2), (B.CAST_F_GRAD_OF_SCALED, 0.5)):
        if rng.random() < p:
            flags |= bit
    compressed = M <= 8 and rng.random() < 0.4
    if compressed:
        flags |= B.CAST_F_EMIT_COMPRESSED
    elif rng.random() < 0.4:
        flags |= B.CAST_F_EMIT_DENSE
    h = Hyper(step=int(rng.integers(1, 500)), total_steps=500)
    ins, states, grads, prevs, tensors = [], [], [], [], []
    for i in range(int(rng.integers(1, 13))):
        n_seg = int(rng.choice([1, 2, 4]))
        seg = max(M, 8) * int(rng.integers(1, 30))
        while (seg * n_seg) % 32:
            seg += max(M, 8)
        rows, cols = int(rng.integers(1, 8)), seg * n_seg
        inp = workloads.gen_tensor_inputs(rows, cols, seed=900 + case, tensor_index=i, scale_mode="jitter")
        gen = torch.Generator().manual_seed(case * 100 + i)
        inp.scale = None if rng.random() < 0.25 else 0.5 + torch.rand((rows, n_seg), generator=gen)
        prev = U.run_oracle(workloads.gen_tensor_inputs(rows, cols, seed=950 + case, tensor_index=i, scale_mode="none"),
                            N, M, Hyper(), RS | (flags & BM))["meta"]
        st = U.to_device(inp, DEV, prev, rows * cols * N // M if compressed else None)
        sg = None
        if inp.scale is not None and rng.random() < 0.7:
            sg = torch.zeros((rows, n_seg), dtype=torch.float32, device=DEV)
        ins.append(inp); states.append(st); grads.append(sg); prevs.append(prev)
        tensors.append(B.make_tensor(st.w.view, st.m.view, st.v.view, st.g.view, st.w_fwd.view, st.meta.view, st.scale,
                                     1 if st.scale is None else n_seg, rows, cols, sg))
    rc, plan = cast.cast_plan_create_ex(tensors, N, M, B.CAST_F_EMIT_COMPRESSED if compressed else 0)
    cast.check(rc)
    flips = torch.zeros(1, dtype=torch.int64, device=DEV)
    lr, b1, b2, eps, lam = h.as_f32()
    cast.check(cast.cast_plan_step(plan, B.make_hyper(lr, b1, b2, eps, lam, h.step, h.total_steps, flags), flips,
                                   torch.cuda.current_stream()))
    torch.cuda.synchronize()
    cast.check(cast.cast_plan_destroy(plan))
    total = 0
    for i, (inp, st, sg, prev) in enumerate(zip(ins, states, grads, prevs)):
        assert st.all_intact()
        ref = U.run_oracle(inp, N, M, h, flags, meta_in=prev)
        got = U.device_outputs(st)
        U.assert_parity(got, ref, f"case {case} tensor {i}: {N}:{M} {inp.w.shape} flags {flags:#x}")
        total += ref["flips"]
        if sg is not None and flags & B.CAST_F_GRAD_OF_SCALED:
            rows, cols = inp.w.shape
            n_seg = inp.scale.shape[1]
            bound = 2e-6 * np.abs(inp.g.double().numpy() * inp.w.double().numpy()).reshape(rows, n_seg, cols // n_seg).sum(-1) + 1e-30
            assert np.all(np.abs(sg.cpu().numpy().astype(np.float64) - ref["scale_grad"]) <= bound)
        elif sg is not None:
            assert float(sg.abs().max().item()) == 0.0            # untouched without the flag
    if flags & B.CAST_F_COUNT_FLIPS:
        assert int(flips.item()) == total


def test_plan_step_replayed_from_a_cuda_graph():
    """A plan step is one kernel launch whose tables travel as parameters, so it can be recorded into a CUDA graph
    and replayed: three replays are three iterations with the recorded hyper-parameters."""
    shapes = [(64, 1056), (7, 2080), (33, 2048)]
    ins = [workloads.gen_tensor_inputs(r, c, seed=27, tensor_index=i, scale_mode="jitter" if c % 64 == 0 else "none")
           for i, (r, c) in enumerate(shapes)]
    states = [U.to_device(inp, DEV) for inp in ins]
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale,
                             1 if s.scale is None else s.scale.shape[1], s.rows, s.cols) for s in states]
    rc, plan = cast.cast_plan_create(tensors, 2, 4)
    cast.check(rc)
    h = Hyper()
    lr, b1, b2, eps, lam = h.as_f32()
    hs = B.make_hyper(lr, b1, b2, eps, lam, h.step, h.total_steps, RS)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        cast.check(cast.cast_plan_step(plan, hs, None, torch.cuda.current_stream()))
    launches = cast.cast_kernel_launch_count()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == launches              # replays launch from the graph, not through the library
    for i, (s, inp) in enumerate(zip(states, ins)):
        cur = inp
        for _ in range(3):
            ref = U.run_oracle(cur, 2, 4, h, RS)
            cur = workloads.TensorInputs(torch.from_numpy(ref["w"]), inp.g, torch.from_numpy(ref["m"]), torch.from_numpy(ref["v"]), inp.scale)
        assert s.all_intact()
        got = U.device_outputs(s)
        # three chained steps: the fp32 state of step k feeds step k + 1, so the comparison is of the last step
        # given slightly different inputs; bounds scale with the step count
        for k in ("w", "m", "v"):
            ok, worst = within_tol(got[k], ref[k], rel=3e-6, floor=3e-9)
            assert ok, f"graph replay tensor {i} {k}: {worst:.3g}"
    cast.check(cast.cast_plan_destroy(plan))


def test_compressed_plan_and_host_step():
    """Plans made for compressed forward-weight buffers, and the host-staged step with the compressed form."""
    shapes = [(3, 96), (64, 1056), (7, 2080), (1, 32)]
    C = B.CAST_F_EMIT_COMPRESSED
    ins = [workloads.gen_tensor_inputs(r, c, seed=26, tensor_index=i, scale_mode="jitter" if c % 64 == 0 else "none")
           for i, (r, c) in enumerate(shapes)]
    for N, M, enc in ((2, 4, 0), (4, 8, BM)):
        states = [U.to_device(inp, DEV, None, inp.w.numel() * N // M) for inp in ins]
        tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, s.scale,
                                 1 if s.scale is None else s.scale.shape[1], s.rows, s.cols) for s in states]
        rc, plan = cast.cast_plan_create_ex(tensors, N, M, C)
        cast.check(rc)
        h = Hyper()
        lr, b1, b2, eps, lam = h.as_f32()
        before = cast.cast_kernel_launch_count()
        # a step without the flag is refused: the buffers are too short for the full form
        assert cast.cast_plan_step(plan, B.make_hyper(lr, b1, b2, eps, lam, h.step, h.total_steps, RS | enc), None, None) == B.CAST_ERR_PLAN
        assert cast.cast_kernel_launch_count() == before
        cast.check(cast.cast_plan_step(plan, B.make_hyper(lr, b1, b2, eps, lam, h.step, h.total_steps, RS | enc | C), None,
                                       torch.cuda.current_stream()))
        torch.cuda.synchronize()
        cast.check(cast.cast_plan_destroy(plan))
        for i, (s, inp) in enumerate(zip(states, ins)):
            assert s.all_intact()
            U.assert_parity(U.device_outputs(s), U.run_oracle(inp, N, M, h, RS | enc | C), f"compressed plan {N}:{M} tensor {i}")
    # an ordinary plan refuses the flag
    states = [U.to_device(inp, DEV) for inp in ins]
    tensors = [B.make_tensor(s.w.view, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, None, 1, s.rows, s.cols) for s in states]
    rc, plan = cast.cast_plan_create(tensors, 2, 4)
    cast.check(rc)
    assert cast.cast_plan_step(plan, B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 1e-3, 1, 10, RS | C), None, None) == B.CAST_ERR_PLAN
    cast.check(cast.cast_plan_destroy(plan))
    # host-resident state, blocks of 4 rows
    rows, cols = 37, 1024
    inp = workloads.gen_tensor_inputs(rows, cols, seed=33, scale_mode="jitter")
    ref = U.run_oracle(inp, 2, 4, Hyper(), RS | C)
    w, m, v, g, sc = pinned(inp.w), pinned(inp.m), pinned(inp.v), pinned(inp.g), pinned(inp.scale)
    fwd = pinned(torch.zeros((rows, cols // 2), dtype=torch.bfloat16))
    meta = pinned(torch.zeros((rows, cols // 32), dtype=torch.int32))
    rc, ctx = cast.cast_host_ctx_create(4096, 2)
    cast.check(rc)
    lr, b1, b2, eps, lam = Hyper().as_f32()
    cast.check(cast.cast_host_step(ctx, w, m, v, g, fwd, meta, sc, 2, rows, cols, 2, 4, lr, b1, b2, eps, lam, 1000, 30000, RS | C, None))
    cast.check(cast.cast_host_ctx_destroy(ctx))
    got = dict(w=w.numpy(), m=m.numpy(), v=v.numpy(), w_fwd=workloads.bf16_bits(fwd), meta=meta.numpy().view(np.uint32))
    U.assert_parity(got, ref, "host blocks, compressed")
    fwd2 = torch.zeros((rows, cols // 2), dtype=torch.bfloat16)
    st2 = [inp.w.clone(), inp.m.clone(), inp.v.clone()]
    meta2 = torch.zeros((rows, cols // 32), dtype=torch.int32)
    cast.check(cast.cast_host_step_static(st2[0], st2[1], st2[2], inp.g, fwd2, meta2, inp.scale, 2, rows, cols, 2, 4,
                                          lr, b1, b2, eps, lam, 1000, 30000, RS | C, None, None))
    got = dict(w=st2[0].numpy(), m=st2[1].numpy(), v=st2[2].numpy(), w_fwd=workloads.bf16_bits(fwd2), meta=meta2.numpy().view(np.uint32))
    U.assert_parity(got, ref, "static staging, compressed")


def test_streamed_layers_on_two_streams_match_oracle():
    """Per-layer plan calls alternating on two streams over fewer resident slots than layers: 6 layers in 4
    slots, so slots 0 and 1 are stepped twice (layers 0, 4 and 1, 5) and slots 2 and 3 once."""
    from paper_2509_25996_b200.runner import StreamedModelState, Hyper as RunHyper
    layer_shapes = [(64, 256), (64, 256), (96, 256), (64, 384)]
    st = StreamedModelState(layer_shapes, n_layers=6, n_slots=4, n_streams=2, N=2, M=4, seed=3, device=DEV,
                            scale_mode="jitter")
    before = [[workloads.TensorInputs(m.w.cpu(), m.g.cpu(), m.m.cpu(), m.v.cpu(), m.scale.cpu()) for m in slot.mats]
              for slot in st.slots]
    h = RunHyper()
    launches = cast.cast_kernel_launch_count()
    st.step(h, RS)
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == launches + 6
    oh = Hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step, h.total_steps)
    for si, slot in enumerate(st.slots):
        for mi, mat in enumerate(slot.mats):
            inp = before[si][mi]
            for _ in range(2 if si < 2 else 1):
                ref = U.run_oracle(inp, 2, 4, oh, RS)
                inp = workloads.TensorInputs(torch.from_numpy(ref["w"]), inp.g, torch.from_numpy(ref["m"]),
                                             torch.from_numpy(ref["v"]), inp.scale)
            got = dict(w=mat.w.cpu().numpy(), m=mat.m.cpu().numpy(), v=mat.v.cpu().numpy(),
                       w_fwd=workloads.bf16_bits(mat.w_fwd), meta=mat.meta.cpu().numpy().view(np.uint32))
            U.assert_parity(got, ref, f"slot {si} matrix {mi}")
    st.close()


def test_plan_rejects_wrong_device_memory_and_survives():
    inp = workloads.gen_tensor_inputs(4, 64, seed=23)
    s = U.to_device(inp, DEV)
    host = torch.zeros(4 * 64)
    bad = B.make_tensor(host, s.m.view, s.v.view, s.g.view, s.w_fwd.view, s.meta.view, None, 1, 4, 64)
    rc, plan = cast.cast_plan_create([bad], 2, 4)
    assert rc == B.CAST_ERR_MEMORY and plan is None


# ------------------------------------------------------------------------------- host-resident state


@pytest.mark.parametrize("block,slots", [(4096, 2), (8192 * 3, 3)])
def test_host_step_blocks_match_oracle(block, slots):
    rows, cols = 37, 1024                      # 37 rows in blocks of 4 (or 24) rows: several blocks + a short one
    inp = workloads.gen_tensor_inputs(rows, cols, seed=30, scale_mode="jitter")
    h = Hyper()
    prev = U.run_oracle(workloads.gen_tensor_inputs(rows, cols, seed=31), 2, 4, h, RS)["meta"]
    fl = RS | B.CAST_F_COUNT_FLIPS
    ref = U.run_oracle(inp, 2, 4, h, fl, meta_in=prev)
    w, m, v, g, sc = pinned(inp.w), pinned(inp.m), pinned(inp.v), pinned(inp.g), pinned(inp.scale)
    fwd = pinned(torch.zeros((rows, cols), dtype=torch.bfloat16))
    meta = pinned(torch.from_numpy(prev.view(np.int32).copy()))
    flips = np.zeros(1, dtype=np.uint64)
    rc, ctx = cast.cast_host_ctx_create(block, slots)
    cast.check(rc)
    lr, b1, b2, eps, lam = h.as_f32()
    cast.check(cast.cast_host_step(ctx, w, m, v, g, fwd, meta, sc, 2, rows, cols, 2, 4, lr, b1, b2, eps, lam,
                                   h.step, h.total_steps, fl, flips))
    cast.check(cast.cast_host_ctx_sync(ctx))
    got = dict(w=w.numpy(), m=m.numpy(), v=v.numpy(), w_fwd=workloads.bf16_bits(fwd),
               meta=meta.numpy().view(np.uint32), flips=int(flips[0]))
    U.assert_parity(got, ref, f"host blocks of {block}")
    # rows longer than a block are refused
    assert cast.cast_host_step(ctx, w, m, v, g, fwd, meta, sc, 2, 1, rows * cols, 2, 4, lr, b1, b2, eps, lam,
                               h.step, h.total_steps, RS, None) in (B.CAST_ERR_PLAN, B.CAST_ERR_SHAPE)
    cast.check(cast.cast_host_ctx_destroy(ctx))


@pytest.mark.parametrize("case", range(10))
def test_random_host_steps(case):
    """Host-resident state through staged blocks (allocated slots and the built-in staging area) with random shapes,
    block sizes, N:M and flags."""
    rng = np.random.default_rng(4000 + case)
    N, M = [(2, 4), (4, 8), (1, 4), (2, 4), (3, 8)][case % 5]
    flags = (RS if rng.random() < 0.8 else 0) | (0 if (N, M) == (2, 4) and rng.random() < 0.5 else BM)
    if rng.random() < 0.5:
        flags |= B.CAST_F_COUNT_FLIPS
    emit = rng.random()
    if emit < 0.3:
        flags |= B.CAST_F_EMIT_COMPRESSED
    elif emit < 0.6:
        flags |= B.CAST_F_EMIT_DENSE
    rows, cols = int(rng.integers(1, 60)), 64 * int(rng.integers(1, 20))
    inp = workloads.gen_tensor_inputs(rows, cols, seed=4100 + case, scale_mode=("jitter" if rng.random() < 0.7 else "none"))
    prev = U.run_oracle(workloads.gen_tensor_inputs(rows, cols, seed=4200 + case, scale_mode="none"), N, M, Hyper(), RS | (flags & BM))["meta"]
    h = Hyper(step=int(rng.integers(1, 100)), total_steps=100)
    ref = U.run_oracle(inp, N, M, h, flags, meta_in=prev)
    lr, b1, b2, eps, lam = h.as_f32()
    fcols = cols * N // M if flags & B.CAST_F_EMIT_COMPRESSED else cols
    n_seg = 1 if inp.scale is None else inp.scale.shape[1]
    block = max(1024, cols * int(rng.integers(1, 8)))
    block += (-block) % 32
    rc, ctx = cast.cast_host_ctx_create(block, int(rng.integers(2, 5)))
    cast.check(rc)
    for which in ("slots", "static"):
        w, m, v = inp.w.clone(), inp.m.clone(), inp.v.clone()
        fwd = torch.zeros((rows, fcols), dtype=torch.bfloat16)
        meta = torch.from_numpy(prev.view(np.int32).copy())
        flips = np.zeros(1, dtype=np.uint64)
        if which == "slots":
            cast.check(cast.cast_host_step(ctx, w, m, v, inp.g, fwd, meta, inp.scale, n_seg, rows, cols, N, M, lr, b1, b2, eps, lam,
                                           h.step, h.total_steps, flags, flips))
            cast.check(cast.cast_host_ctx_sync(ctx))
        else:
            cast.check(cast.cast_host_step_static(w, m, v, inp.g, fwd, meta, inp.scale, n_seg, rows, cols, N, M, lr, b1, b2, eps, lam,
                                                  h.step, h.total_steps, flags, flips, None))
        got = dict(w=w.numpy(), m=m.numpy(), v=v.numpy(), w_fwd=workloads.bf16_bits(fwd), meta=meta.numpy().view(np.uint32))
        if flags & B.CAST_F_COUNT_FLIPS:
            got["flips"] = int(flips[0])
        U.assert_parity(got, ref, f"case {case} {which}: {N}:{M} {rows}x{cols} block {block} flags {flags:#x}")
    cast.check(cast.cast_host_ctx_destroy(ctx))


def test_host_step_pageable_memory():
    rows, cols = 8, 512
    inp = workloads.gen_tensor_inputs(rows, cols, seed=32, scale_mode="none")
    ref = U.run_oracle(inp, 2, 4, Hyper(), RS)
    fwd = torch.zeros((rows, cols), dtype=torch.bfloat16)
    meta = torch.zeros((rows, cols // 32), dtype=torch.int32)
    rc, ctx = cast.cast_host_ctx_create(2048, 2)
    cast.check(rc)
    lr, b1, b2, eps, lam = Hyper().as_f32()
    cast.check(cast.cast_host_step(ctx, inp.w, inp.m, inp.v, inp.g, fwd, meta, None, 1, rows, cols, 2, 4,
                                   lr, b1, b2, eps, lam, 1000, 30000, RS, None))
    cast.check(cast.cast_host_ctx_destroy(ctx))
    got = dict(w=inp.w.numpy(), m=inp.m.numpy(), v=inp.v.numpy(), w_fwd=workloads.bf16_bits(fwd),
               meta=meta.numpy().view(np.uint32))
    U.assert_parity(got, ref, "pageable")


def test_plan_access_paths_give_the_same_bits():
    """A plan step takes the staged access path where it is built unless told otherwise: the default, the forced staged
    and the forced plain launches of the same steps agree bit for bit, flips included, and no staged wait ran out."""
    from paper_2509_25996_b200.runner import DeviceModelState, Hyper as RunHyper
    shapes = [(24, 256), (7, 2080), (3, 1056), (4096, 4096), (40, 512)]         # 16.8 M parameters: above the size from which
    paths = (0, B.CAST_F_BULK_STAGING, B.CAST_F_PLAIN_ACCESS)                   # a plan stages by default
    states = [DeviceModelState(shapes, 2, 4, seed=6, device="cuda:0", scale_mode="jitter") for _ in paths]
    h = RunHyper(total_steps=30000)
    launches = cast.cast_kernel_launch_count()
    for flags in (B.CAST_F_RESELECT, B.CAST_F_EMIT_DENSE, B.CAST_F_RESELECT | B.CAST_F_COUNT_FLIPS | B.CAST_F_EMIT_DENSE):
        for st, path in zip(states, paths):
            st.step(h, flags | path)
        h.step += 1
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == launches + 9
    for other in states[1:]:
        for x, y in zip(states[0].mats, other.mats):
            for k in ("w", "m", "v", "w_fwd", "meta"):
                assert torch.equal(getattr(x, k), getattr(y, k)), k
        assert int(other.flips.item()) == int(states[0].flips.item()) > 0
    rc, timeouts = cast.cast_bulk_timeout_count()
    assert rc == 0 and timeouts == 0
    # a configuration the staged path is not built for runs plain by default and is refused when staged is forced
    hy = B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 1e-3, h.step, 30000, B.CAST_F_RESELECT | B.CAST_F_V_KEPT_FROM_G)
    cast.check(cast.cast_plan_step(states[0].plan, hy, None, None))
    hy.flags |= B.CAST_F_BULK_STAGING
    assert cast.cast_plan_step(states[0].plan, hy, None, None) == B.CAST_ERR_NM
    torch.cuda.synchronize()
    for st in states:
        st.close()


def test_a_plan_that_gave_up_on_a_staged_copy_refuses_further_steps():
    """The staged kernels wait for their copies a bounded time; a tile they give up on is reported in a word of host
    memory the plan owns, and the plan then answers CAST_ERR_STAGING instead of stepping on over a state that was not
    fully updated.  The report is injected on the host here (no GPU wait is made to run out)."""
    from paper_2509_25996_b200.runner import DeviceModelState, Hyper as RunHyper
    st = DeviceModelState([(16, 512)], 2, 4, seed=9, device="cuda:0", scale_mode="ones")
    h = RunHyper(total_steps=30000)
    st.step(h, B.CAST_F_RESELECT)
    torch.cuda.synchronize()
    launches = cast.cast_kernel_launch_count()
    assert cast.cast_plan_report_staging_failure(st.plan) == B.CAST_OK
    hy = B.make_hyper(h.lr, h.beta1, h.beta2, h.eps, h.l1_coeff, h.step + 1, h.total_steps, B.CAST_F_RESELECT)
    assert cast.cast_plan_step(st.plan, hy, None, None) == B.CAST_ERR_STAGING
    hy.flags |= B.CAST_F_PLAIN_ACCESS
    assert cast.cast_plan_step(st.plan, hy, None, None) == B.CAST_ERR_STAGING          # whatever the path
    assert cast.cast_kernel_launch_count() == launches
    assert "bulk copy" in cast.cast_strerror(B.CAST_ERR_STAGING)
    assert cast.cast_plan_report_staging_failure(None) == B.CAST_ERR_PLAN
    st.close()
