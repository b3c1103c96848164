"""cast_host_step_static: the host-resident AdamS step for callers that must not allocate device memory.

Some users of this library cannot call cudaMalloc when they step the optimizer: their framework's
allocator already owns the whole device, or they run where the device-wide synchronisation of an
allocation is not acceptable.  For them the library carries its own staging area (a fixed array in the
library image).  This test calls that entry point through the C ABI and checks that it gives what the
allocating entry point (cast_host_step) gives on the same inputs -- twice in a row, with a different
shape, flags and metadata form the second time, because every call reuses the same area and must not see
what the previous call left there -- and that the second call leaves the amount of free device memory
untouched (the first call on a device is the one that may bring the library's device image in, which is why
such callers make it at start-up).  The file name sorts last so that a run that stops at the first
failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle.adams_oracle import Hyper
import gpu_util as U

pytestmark = pytest.mark.gpu

RS, BM, FL = B.CAST_F_RESELECT, B.CAST_F_META_BITMASK, B.CAST_F_COUNT_FLIPS


def host_state(rows, cols, seed, meta_in):
    inp = workloads.gen_tensor_inputs(rows, cols, seed=seed, scale_mode="jitter")
    return dict(w=inp.w.clone(), m=inp.m.clone(), v=inp.v.clone(), g=inp.g.clone(), scale=inp.scale.clone(),
                fwd=torch.zeros((rows, cols), dtype=torch.bfloat16),
                meta=torch.from_numpy(meta_in.view(np.int32).copy()), flips=np.zeros(1, dtype=np.uint64), inp=inp)


def outputs(st):
    return dict(w=st["w"].numpy(), m=st["m"].numpy(), v=st["v"].numpy(), w_fwd=workloads.bf16_bits(st["fwd"]),
                meta=st["meta"].numpy().view(np.uint32), flips=int(st["flips"][0]))


def step_with_context(st, rows, cols, N, M, h, flags):
    """The existing entry point: staging slots allocated by cast_host_ctx_create."""
    rc, ctx = cast.cast_host_ctx_create(8192, 2)
    cast.check(rc)
    lr, b1, b2, eps, lam = h.as_f32()
    cast.check(cast.cast_host_step(ctx, st["w"], st["m"], st["v"], st["g"], st["fwd"], st["meta"], st["scale"], 2,
                                   rows, cols, N, M, lr, b1, b2, eps, lam, h.step, h.total_steps, flags, st["flips"]))
    cast.check(cast.cast_host_ctx_destroy(ctx))


def step_static(st, rows, cols, N, M, h, flags, stream=None):
    lr, b1, b2, eps, lam = h.as_f32()
    return cast.cast_host_step_static(st["w"], st["m"], st["v"], st["g"], st["fwd"], st["meta"], st["scale"], 2,
                                      rows, cols, N, M, lr, b1, b2, eps, lam, h.step, h.total_steps, flags,
                                      st["flips"], stream)


def test_static_staging_matches_allocating_entry_point_on_two_calls_in_a_row():
    torch.cuda.set_device(0)
    h = Hyper()
    calls = [
        # a larger matrix first, index-form 2:4 metadata, flips counted against another matrix's mask
        dict(rows=37, cols=1024, N=2, M=4, flags=RS | FL, seed=40),
        # then a smaller one with 4:8 bitmask metadata: whatever the first call left must not show
        dict(rows=5, cols=512, N=4, M=8, flags=RS | BM | FL, seed=41),
    ]
    side = torch.cuda.Stream()
    for i, c in enumerate(calls):
        rows, cols, N, M, flags = c["rows"], c["cols"], c["N"], c["M"], c["flags"]
        enc = flags & BM
        prev = U.run_oracle(workloads.gen_tensor_inputs(rows, cols, seed=c["seed"] + 10), N, M, h, RS | enc)["meta"]
        a = host_state(rows, cols, c["seed"], prev)
        b = host_state(rows, cols, c["seed"], prev)
        step_with_context(a, rows, cols, N, M, h, flags)
        launches = cast.cast_kernel_launch_count()
        free_before, _ = torch.cuda.mem_get_info()
        cast.check(step_static(b, rows, cols, N, M, h, flags, stream=(side if i else None)))
        free_after, _ = torch.cuda.mem_get_info()
        assert cast.cast_kernel_launch_count() == launches + 1
        if i:
            # The first call on a device may load the part of the library that holds the staging area (CUDA loads
            # device code lazily); every later call must leave the amount of free device memory exactly as it was.
            assert free_after == free_before, f"the call changed free device memory by {free_before - free_after} bytes"
        got, want = outputs(b), outputs(a)
        U.assert_parity(got, want, f"call {i}: static staging vs allocated staging")
        assert got["flips"] == want["flips"] > 0
        # and both agree with the CPU oracle
        U.assert_parity(got, U.run_oracle(a["inp"], N, M, h, flags, meta_in=prev), f"call {i}: static staging vs oracle")


def test_static_staging_refuses_matrices_beyond_its_size():
    torch.cuda.set_device(0)
    rows, cols = 1025, 1024                       # 1,049,600 parameters > CAST_STATIC_MAX_PARAMS
    assert rows * cols > B.CAST_STATIC_MAX_PARAMS
    st = dict(w=torch.zeros(rows, cols), m=torch.zeros(rows, cols), v=torch.zeros(rows, cols),
              g=torch.zeros(rows, cols, dtype=torch.bfloat16), scale=torch.ones(rows, 2),
              fwd=torch.zeros(rows, cols, dtype=torch.bfloat16), meta=torch.zeros(rows, cols // 32, dtype=torch.int32),
              flips=np.zeros(1, dtype=np.uint64))
    before = cast.cast_kernel_launch_count()
    rc = step_static(st, rows, cols, 2, 4, Hyper(), RS)
    assert rc == B.CAST_ERR_PLAN and cast.cast_kernel_launch_count() == before
    # the largest size it takes: exactly the limit
    rows = B.CAST_STATIC_MAX_PARAMS // cols
    inp = workloads.gen_tensor_inputs(rows, cols, seed=42, scale_mode="jitter")
    st = dict(w=inp.w.clone(), m=inp.m.clone(), v=inp.v.clone(), g=inp.g, scale=inp.scale,
              fwd=torch.zeros(rows, cols, dtype=torch.bfloat16), meta=torch.zeros(rows, cols // 32, dtype=torch.int32),
              flips=np.zeros(1, dtype=np.uint64))
    cast.check(step_static(st, rows, cols, 2, 4, Hyper(), RS))
    U.assert_parity({k: v for k, v in outputs(st).items() if k != "flips"}, U.run_oracle(inp, 2, 4, Hyper(), RS), "at the size limit")
