"""The C-ABI library: it loads, exports what the header declares, and rejects bad arguments on the
host without launching anything.  No test here needs a GPU (fake, never-dereferenced addresses)."""
import ctypes
import os
import re

import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _lib():
    import __graft_entry__
    __graft_entry__.build()


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"CAST_API\s+[\w\s\*]+?\b(cast_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    lib = B.load_library()
    names = declared_functions()
    assert len(names) >= 11 and set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_strerror_covers_all_statuses():
    for s in range(0, -11, -1):
        assert cast.cast_strerror(s) != "unknown status"
    assert cast.cast_strerror(-99) == "unknown status"


# fake device addresses: 16-byte aligned, far apart, never dereferenced because validation fails first
W, M_, V, G, F, META, SC = (0x10000000 * k for k in range(1, 8))
GOOD = dict(w=W, m=M_, v=V, g=G, w_fwd_bf16=F, meta=META, scale=None, scale_groups=1, rows=4, cols=64, N=2, M=4,
            lr=1e-4, beta1=0.9, beta2=0.95, eps=1e-8, l1_coeff=1e-3, step=10, total_steps=100,
            flags=B.CAST_F_RESELECT, flip_count=None, stream=None)


def call(**over):
    a = dict(GOOD)
    a.update(over)
    return cast.cast_adams_step(**a)


@pytest.mark.parametrize("over,status", [
    (dict(w=None), B.CAST_ERR_NULL),
    (dict(g=None), B.CAST_ERR_NULL),
    (dict(meta=None), B.CAST_ERR_NULL),
    (dict(flags=B.CAST_F_RESELECT | B.CAST_F_COUNT_FLIPS), B.CAST_ERR_NULL),          # flip_count missing
    (dict(cols=48), B.CAST_ERR_SHAPE),                                                  # cols % 32
    (dict(rows=0), B.CAST_ERR_SHAPE),
    (dict(rows=1 << 20, cols=1 << 12), B.CAST_ERR_SHAPE),                               # rows*cols >= 2^31
    (dict(scale=SC, scale_groups=3), B.CAST_ERR_SHAPE),                                 # 64 % 3
    (dict(scale=SC, scale_groups=16), B.CAST_ERR_SHAPE),                                # 4-column segments < unit
    (dict(scale=SC, scale_groups=0), B.CAST_ERR_SHAPE),
    (dict(m=M_ + 4), B.CAST_ERR_ALIGN),
    (dict(w_fwd_bf16=F + 2), B.CAST_ERR_ALIGN),
    (dict(N=3, M=4), B.CAST_ERR_NM),                                                    # index form is 2:4 only
    (dict(N=0, M=4, flags=B.CAST_F_RESELECT | B.CAST_F_META_BITMASK), B.CAST_ERR_NM),
    (dict(N=5, M=4, flags=B.CAST_F_RESELECT | B.CAST_F_META_BITMASK), B.CAST_ERR_NM),
    (dict(N=2, M=6, flags=B.CAST_F_RESELECT | B.CAST_F_META_BITMASK), B.CAST_ERR_NM),
    (dict(N=2, M=64, flags=B.CAST_F_RESELECT | B.CAST_F_META_BITMASK), B.CAST_ERR_NM),
    (dict(step=0), B.CAST_ERR_HYPER),
    (dict(step=101), B.CAST_ERR_HYPER),
    (dict(beta1=1.0), B.CAST_ERR_HYPER),
    (dict(beta2=-0.1), B.CAST_ERR_HYPER),
    (dict(eps=0.0), B.CAST_ERR_HYPER),
    (dict(lr=float("nan")), B.CAST_ERR_HYPER),
    (dict(l1_coeff=float("inf")), B.CAST_ERR_HYPER),
    (dict(flags=1 << 10), B.CAST_ERR_HYPER),                                            # unknown flag bit
    (dict(flags=B.CAST_F_RESELECT | B.CAST_F_BULK_STAGING | B.CAST_F_PLAIN_ACCESS), B.CAST_ERR_HYPER),
    (dict(m=W + 64), B.CAST_ERR_ALIAS),
    (dict(meta=F + 16), B.CAST_ERR_ALIAS),
])
def test_bad_arguments_are_rejected_before_any_launch(over, status):
    before = cast.cast_kernel_launch_count()
    assert call(**over) == status
    assert cast.cast_kernel_launch_count() == before


def test_wellformed_call_without_device_memory_fails_cleanly():
    """Fake addresses that pass every host rule: with no driver the runtime call fails (CAST_ERR_CUDA);
    with a driver the addresses are recognised as not being device memory (CAST_ERR_MEMORY)."""
    before = cast.cast_kernel_launch_count()
    rc = call()
    assert rc in (B.CAST_ERR_CUDA, B.CAST_ERR_MEMORY)
    if rc == B.CAST_ERR_CUDA:
        assert cast.cast_last_cuda_error() != 0
    assert cast.cast_kernel_launch_count() == before
    with pytest.raises(cast.CastError):
        cast.check(rc)


def test_plan_argument_checks():
    t = B.make_tensor(W, M_, V, G, F, META, None, 1, 4, 64)
    assert cast.cast_plan_create([], 2, 4)[0] == B.CAST_ERR_NULL                # no descriptor array at all
    assert cast.cast_plan_create([t], 2, 5)[0] == B.CAST_ERR_NM
    bad = B.make_tensor(W, M_, V, G, F, META, None, 1, 4, 40)
    assert cast.cast_plan_create([t, bad], 2, 4)[0] == B.CAST_ERR_SHAPE
    bad = B.make_tensor(W, None, V, G, F, META, None, 1, 4, 64)
    assert cast.cast_plan_create([bad], 2, 4)[0] == B.CAST_ERR_NULL
    rc, plan = cast.cast_plan_create([t], 2, 4)
    assert rc in (B.CAST_ERR_CUDA, B.CAST_ERR_MEMORY) and plan is None
    assert cast.cast_plan_step(None, B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 0, 1, 1, 1)) == B.CAST_ERR_PLAN
    assert cast.cast_plan_destroy(None) == B.CAST_ERR_PLAN
    # a handle that is not a plan (readable memory with the wrong signature)
    junk = ctypes.create_string_buffer(256)
    assert cast.cast_plan_step(ctypes.addressof(junk), B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 0, 1, 1, 1)) == B.CAST_ERR_PLAN
    assert cast.cast_plan_destroy(ctypes.addressof(junk)) == B.CAST_ERR_PLAN


def test_host_context_argument_checks():
    assert cast.cast_host_ctx_create(1000, 2)[0] == B.CAST_ERR_SHAPE          # not a multiple of 32 / too small
    assert cast.cast_host_ctx_create(1 << 20, 1)[0] == B.CAST_ERR_SHAPE
    assert cast.cast_host_ctx_create(1 << 20, 9)[0] == B.CAST_ERR_SHAPE
    assert cast.cast_host_ctx_sync(None) == B.CAST_ERR_PLAN
    assert cast.cast_host_ctx_destroy(None) == B.CAST_ERR_PLAN
    junk = ctypes.create_string_buffer(1024)
    assert cast.cast_host_step(ctypes.addressof(junk), W, M_, V, G, F, META, None, 1, 4, 64, 2, 4,
                               1e-4, 0.9, 0.95, 1e-8, 1e-3, 1, 10, B.CAST_F_RESELECT) == B.CAST_ERR_PLAN
    if not torch.cuda.is_available():
        rc, ctx = cast.cast_host_ctx_create(1 << 20, 2)
        assert rc == B.CAST_ERR_CUDA and ctx is None


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libcast_adams.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.load_library()


def test_mask_stats_argument_checks():
    ok = dict(w=W, meta=META, meta_ref=None, rows=4, cols=64, M=4, flags=0, stats=SC)
    def call_stats(**over):
        a = dict(ok); a.update(over)
        return cast.cast_mask_stats(**a)
    before = cast.cast_kernel_launch_count()
    assert call_stats(w=None) == B.CAST_ERR_NULL
    assert call_stats(stats=None) == B.CAST_ERR_NULL
    assert call_stats(M=3) == B.CAST_ERR_NM
    assert call_stats(M=8) == B.CAST_ERR_NM                       # index form is 2:4 only
    assert call_stats(flags=B.CAST_F_RESELECT) == B.CAST_ERR_HYPER
    assert call_stats(cols=48) == B.CAST_ERR_SHAPE
    assert call_stats(meta=META + 4) == B.CAST_ERR_ALIGN
    assert call_stats(stats=SC + 4) == B.CAST_ERR_ALIGN
    assert call_stats() in (B.CAST_ERR_CUDA, B.CAST_ERR_MEMORY)   # fake addresses are not device memory
    assert cast.cast_kernel_launch_count() == before


def test_later_entry_points_check_their_arguments_without_a_gpu():
    """Every check that needs no device runs before the first CUDA call, so these hold on a machine without a GPU."""
    before = cast.cast_kernel_launch_count()
    # final pruning
    assert cast.cast_prune_fold(None, None, 1, META, F, 4, 64, 2, 4, B.CAST_F_RESELECT) == B.CAST_ERR_NULL
    assert cast.cast_prune_fold(W, None, 1, META, F, 4, 64, 3, 8, B.CAST_F_RESELECT) == B.CAST_ERR_NM
    assert cast.cast_prune_fold(W, None, 1, META, F, 4, 64, 2, 4, B.CAST_F_EMIT_DENSE) == B.CAST_ERR_HYPER
    assert cast.cast_prune_fold(W, None, 1, META, F + 2, 4, 64, 2, 4, B.CAST_F_RESELECT) == B.CAST_ERR_ALIGN
    assert cast.cast_prune_fold(W, None, 1, META, W + 64, 4, 64, 2, 4, B.CAST_F_RESELECT) == B.CAST_ERR_ALIAS
    assert cast.cast_plan_prune_fold(None, None, B.CAST_F_RESELECT) == B.CAST_ERR_PLAN
    # distillation loss
    assert cast.cast_kd_loss(W, M_, None, V, None, 4, 64, 0.5) == B.CAST_ERR_NULL
    assert cast.cast_kd_loss(W, M_, G, V, None, 4, 0, 0.5) == B.CAST_ERR_SHAPE
    assert cast.cast_kd_loss(W, M_, G, V, None, 4, 64, -0.1) == B.CAST_ERR_HYPER
    assert cast.cast_kd_loss(W, M_, G, V, None, 4, 64, 0.5, float("inf")) == B.CAST_ERR_HYPER
    assert cast.cast_kd_loss(W + 1, M_, G, V, None, 4, 64, 0.5) == B.CAST_ERR_ALIGN
    assert cast.cast_kd_loss(W, M_, G, V, W + 128, 4, 64, 0.5) == B.CAST_ERR_ALIAS
    # scale training
    assert cast.cast_scale_adam_step(W, M_, V, None, 8, 1e-3, 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_NULL
    assert cast.cast_scale_adam_step(W, M_, V, G, 8, float("nan"), 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_HYPER
    assert cast.cast_scale_adam_step(W, W + 16, V, G, 8, 1e-3, 0.9, 0.95, 1e-8, 1) == B.CAST_ERR_ALIAS
    hyper = B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 1e-3, 10, 100, B.CAST_F_RESELECT)
    t = B.make_tensor(W, M_, V, G, F, META, None, 1, 4, 64)
    assert cast.cast_adams_step_ex(None, 2, 4, hyper) == B.CAST_ERR_NULL
    assert cast.cast_adams_step_ex(t, 2, 4, None) == B.CAST_ERR_NULL
    assert cast.cast_adams_step_ex(t, 5, 4, hyper) == B.CAST_ERR_NM
    bad = B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 1e-3, 10, 100, B.CAST_F_RESELECT | B.CAST_F_EMIT_DENSE | B.CAST_F_EMIT_COMPRESSED)
    assert cast.cast_adams_step_ex(t, 2, 4, bad) == B.CAST_ERR_HYPER
    wide = B.make_hyper(1e-4, 0.9, 0.95, 1e-8, 1e-3, 10, 100, B.CAST_F_RESELECT | B.CAST_F_META_BITMASK | B.CAST_F_EMIT_COMPRESSED)
    assert cast.cast_adams_step_ex(t, 8, 16, wide) == B.CAST_ERR_NM                   # compressed form needs M <= 8
    huge_lr = B.make_hyper(3e38, 0.9, 0.95, 1e-8, 1e-3, 10, 100, B.CAST_F_RESELECT)
    assert cast.cast_adams_step_ex(t, 2, 4, huge_lr) == B.CAST_ERR_HYPER              # 2^32 lr / bc1 is not a float
    rc, plan = cast.cast_plan_create_ex([t], 2, 4, B.CAST_F_RESELECT)
    assert rc == B.CAST_ERR_HYPER and plan is None                                    # only the compressed flag is a plan property
    rc, plan = cast.cast_plan_create_ex([t], 8, 16, B.CAST_F_EMIT_COMPRESSED)
    assert rc == B.CAST_ERR_NM and plan is None
    # the static staging entry point refuses oversize matrices before touching CUDA
    big_rows = B.CAST_STATIC_MAX_PARAMS // 64 + 1
    assert cast.cast_host_step_static(W, M_, V, G, F, META, None, 1, big_rows, 64, 2, 4, 1e-4, 0.9, 0.95, 1e-8, 1e-3, 1, 10,
                                      B.CAST_F_RESELECT) == B.CAST_ERR_PLAN
    assert cast.cast_kernel_launch_count() == before
