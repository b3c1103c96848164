"""ctypes binding of libcast_adams.so: the same names as the C ABI, argument marshalling only.

Every function returns the library's integer status (0 = CAST_OK); `check()` turns a
non-zero status into a CastError.  Pointer arguments accept a torch tensor, a numpy
array, an integer address or None.  There is no fallback: if the shared library has
not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libcast_adams.so")

# status codes
CAST_OK = 0
CAST_ERR_NULL = -1
CAST_ERR_SHAPE = -2
CAST_ERR_ALIGN = -3
CAST_ERR_NM = -4
CAST_ERR_HYPER = -5
CAST_ERR_CUDA = -6
CAST_ERR_PLAN = -7
CAST_ERR_ALIAS = -8
CAST_ERR_MEMORY = -9
CAST_ERR_STAGING = -10

# flags
CAST_F_RESELECT = 1 << 0
CAST_F_COUNT_FLIPS = 1 << 1
CAST_F_META_BITMASK = 1 << 2
CAST_F_V_KEPT_FROM_G = 1 << 3
CAST_F_EMIT_DENSE = 1 << 4
CAST_F_EMIT_COMPRESSED = 1 << 5
CAST_F_GRAD_OF_SCALED = 1 << 6
CAST_F_MASK_STATS = 1 << 7
CAST_F_BULK_STAGING = 1 << 8
CAST_F_PLAIN_ACCESS = 1 << 9

EXPORTS = (
    "cast_adams_step", "cast_adams_step_ex", "cast_scale_adam_step", "cast_plan_scale_adam_step",
    "cast_plan_create", "cast_plan_create_ex", "cast_plan_step", "cast_plan_step_stats", "cast_plan_destroy", "cast_plan_report_staging_failure",
    "cast_host_ctx_create", "cast_host_step", "cast_host_ctx_sync", "cast_host_ctx_destroy",
    "cast_host_step_static", "cast_kd_loss", "cast_prune_fold", "cast_plan_prune_fold", "cast_mask_stats", "cast_plan_mask_stats",
    "cast_probe_launch", "cast_probe_stream", "cast_bulk_timeout_count",
    "cast_strerror", "cast_last_cuda_error", "cast_kernel_launch_count",
)


class CastError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"cast_adams status {status}: {message}")
        self.status = status


class cast_tensor_t(ctypes.Structure):
    _fields_ = [
        ("w", ctypes.c_void_p), ("m", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("g", ctypes.c_void_p), ("w_fwd", ctypes.c_void_p), ("meta", ctypes.c_void_p),
        ("scale", ctypes.c_void_p), ("scale_groups", ctypes.c_int32),
        ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
        ("scale_grad", ctypes.c_void_p),
        ("meta_ref", ctypes.c_void_p),
        ("scale_chain", ctypes.c_void_p),
    ]


class cast_hyper_t(ctypes.Structure):
    _fields_ = [
        ("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
        ("eps", ctypes.c_float), ("l1_coeff", ctypes.c_float),
        ("step", ctypes.c_int64), ("total_steps", ctypes.c_int64), ("flags", ctypes.c_uint32),
    ]


_lib = None

_STEP_ARGS = [
    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,      # w m v g
    ctypes.c_void_p, ctypes.c_void_p,                                        # w_fwd meta
    ctypes.c_void_p, ctypes.c_int,                                           # scale scale_groups
    ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,              # rows cols N M
    ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_float,
    ctypes.c_int64, ctypes.c_int64,                                          # step total_steps
    ctypes.c_uint32, ctypes.c_void_p,                                        # flags flip_count
]


def load_library() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (there is no other path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2509_25996_b200.build_ext` "
            "(this package has no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.cast_adams_step.restype = ctypes.c_int
    lib.cast_adams_step.argtypes = _STEP_ARGS + [ctypes.c_void_p]
    lib.cast_adams_step_ex.restype = ctypes.c_int
    lib.cast_adams_step_ex.argtypes = [ctypes.POINTER(cast_tensor_t), ctypes.c_int, ctypes.c_int, ctypes.POINTER(cast_hyper_t),
                                       ctypes.c_void_p, ctypes.c_void_p]
    lib.cast_scale_adam_step.restype = ctypes.c_int
    lib.cast_scale_adam_step.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int64, ctypes.c_float, ctypes.c_float, ctypes.c_float,
                                                                 ctypes.c_float, ctypes.c_int64, ctypes.c_int, ctypes.c_void_p]
    lib.cast_plan_scale_adam_step.restype = ctypes.c_int
    lib.cast_plan_scale_adam_step.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p),
                                              ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_int64,
                                              ctypes.c_int, ctypes.c_void_p]
    lib.cast_plan_create.restype = ctypes.c_int
    lib.cast_plan_create.argtypes = [ctypes.POINTER(cast_tensor_t), ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                     ctypes.POINTER(ctypes.c_void_p)]
    lib.cast_plan_create_ex.restype = ctypes.c_int
    lib.cast_plan_create_ex.argtypes = [ctypes.POINTER(cast_tensor_t), ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_uint32,
                                        ctypes.POINTER(ctypes.c_void_p)]
    lib.cast_plan_step.restype = ctypes.c_int
    lib.cast_plan_step.argtypes = [ctypes.c_void_p, ctypes.POINTER(cast_hyper_t), ctypes.c_void_p, ctypes.c_void_p]
    lib.cast_plan_step_stats.restype = ctypes.c_int
    lib.cast_plan_step_stats.argtypes = [ctypes.c_void_p, ctypes.POINTER(cast_hyper_t), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.cast_plan_report_staging_failure.restype = ctypes.c_int
    lib.cast_plan_report_staging_failure.argtypes = [ctypes.c_void_p]
    lib.cast_plan_destroy.restype = ctypes.c_int
    lib.cast_plan_destroy.argtypes = [ctypes.c_void_p]
    lib.cast_host_ctx_create.restype = ctypes.c_int
    lib.cast_host_ctx_create.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p)]
    lib.cast_host_step.restype = ctypes.c_int
    lib.cast_host_step.argtypes = [ctypes.c_void_p] + _STEP_ARGS
    lib.cast_host_step_static.restype = ctypes.c_int
    lib.cast_host_step_static.argtypes = _STEP_ARGS + [ctypes.c_void_p]
    lib.cast_kd_loss.restype = ctypes.c_int
    lib.cast_kd_loss.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int64, ctypes.c_int64, ctypes.c_float, ctypes.c_float, ctypes.c_void_p]
    lib.cast_prune_fold.restype = ctypes.c_int
    lib.cast_prune_fold.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_uint32, ctypes.c_void_p]
    lib.cast_plan_prune_fold.restype = ctypes.c_int
    lib.cast_plan_prune_fold.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_uint32, ctypes.c_void_p]
    lib.cast_mask_stats.restype = ctypes.c_int
    lib.cast_mask_stats.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p]
    lib.cast_plan_mask_stats.restype = ctypes.c_int
    lib.cast_plan_mask_stats.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_uint32, ctypes.c_void_p,
                                         ctypes.c_void_p]
    lib.cast_bulk_timeout_count.restype = ctypes.c_int
    lib.cast_bulk_timeout_count.argtypes = [ctypes.POINTER(ctypes.c_ulonglong)]
    lib.cast_probe_launch.restype = ctypes.c_int
    lib.cast_probe_launch.argtypes = [ctypes.c_int64, ctypes.c_void_p]
    lib.cast_probe_stream.restype = ctypes.c_int
    lib.cast_probe_stream.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int64, ctypes.c_void_p]
    lib.cast_host_ctx_sync.restype = ctypes.c_int
    lib.cast_host_ctx_sync.argtypes = [ctypes.c_void_p]
    lib.cast_host_ctx_destroy.restype = ctypes.c_int
    lib.cast_host_ctx_destroy.argtypes = [ctypes.c_void_p]
    lib.cast_strerror.restype = ctypes.c_char_p
    lib.cast_strerror.argtypes = [ctypes.c_int]
    lib.cast_last_cuda_error.restype = ctypes.c_int
    lib.cast_last_cuda_error.argtypes = []
    lib.cast_kernel_launch_count.restype = ctypes.c_ulonglong
    lib.cast_kernel_launch_count.argtypes = []
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(f"cannot take the address of {type(x)!r}")


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream          # torch.cuda.Stream


def kernel_flag_word(flags: int) -> int:
    """The template argument that names the step kernel a flag word runs (flip counting is dropped where the mask
    is reused: nothing can flip).  Names only; the library picks the kernel itself."""
    f = int(flags) & 0xFF
    if not f & CAST_F_RESELECT:
        f &= ~CAST_F_COUNT_FLIPS
    return f


def cast_strerror(status: int) -> str:
    return load_library().cast_strerror(int(status)).decode()


def cast_last_cuda_error() -> int:
    return int(load_library().cast_last_cuda_error())


def cast_kernel_launch_count() -> int:
    return int(load_library().cast_kernel_launch_count())


def check(status: int) -> None:
    if status != CAST_OK:
        msg = cast_strerror(status)
        if status == CAST_ERR_CUDA:
            msg += f" (cudaError {cast_last_cuda_error()})"
        raise CastError(status, msg)


def cast_adams_step(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols, N, M,
                    lr, beta1, beta2, eps, l1_coeff, step, total_steps, flags, flip_count=None, stream=None) -> int:
    return load_library().cast_adams_step(
        _ptr(w), _ptr(m), _ptr(v), _ptr(g), _ptr(w_fwd_bf16), _ptr(meta), _ptr(scale), int(scale_groups),
        int(rows), int(cols), int(N), int(M), lr, beta1, beta2, eps, l1_coeff, int(step), int(total_steps),
        int(flags), _ptr(flip_count), _stream(stream))


def cast_plan_scale_adam_step(plan, m_as, v_as, lr, beta1, beta2, eps, step, clear_grad=True, stream=None) -> int:
    """`m_as`, `v_as`: sequences of one moment buffer per matrix of the plan."""
    pm = None if m_as is None else (ctypes.c_void_p * len(m_as))(*[_ptr(x) for x in m_as])
    pv = None if v_as is None else (ctypes.c_void_p * len(v_as))(*[_ptr(x) for x in v_as])
    return load_library().cast_plan_scale_adam_step(plan, pm, pv, lr, beta1, beta2, eps, int(step), 1 if clear_grad else 0,
                                                    _stream(stream))


def make_tensor(w, m, v, g, w_fwd, meta, scale, scale_groups, rows, cols, scale_grad=None, meta_ref=None,
                scale_chain=None) -> cast_tensor_t:
    return cast_tensor_t(_ptr(w), _ptr(m), _ptr(v), _ptr(g), _ptr(w_fwd), _ptr(meta), _ptr(scale),
                         int(scale_groups), int(rows), int(cols), _ptr(scale_grad), _ptr(meta_ref), _ptr(scale_chain))


def cast_adams_step_ex(tensor: Optional[cast_tensor_t], N: int, M: int, hyper: Optional[cast_hyper_t],
                       flip_count=None, stream=None) -> int:
    t = ctypes.byref(tensor) if tensor is not None else None
    h = ctypes.byref(hyper) if hyper is not None else None
    return load_library().cast_adams_step_ex(t, int(N), int(M), h, _ptr(flip_count), _stream(stream))


def cast_scale_adam_step(a, m_a, v_a, grad, n, lr, beta1, beta2, eps, step, clear_grad=True, stream=None) -> int:
    return load_library().cast_scale_adam_step(_ptr(a), _ptr(m_a), _ptr(v_a), _ptr(grad), int(n), lr, beta1, beta2, eps,
                                               int(step), 1 if clear_grad else 0, _stream(stream))


def cast_plan_create(tensors: Sequence[cast_tensor_t], N: int, M: int):
    """Returns (status, plan handle or None)."""
    n = len(tensors)
    arr = (cast_tensor_t * max(n, 1))(*tensors)
    out = ctypes.c_void_p(None)
    rc = load_library().cast_plan_create(arr if n else None, n, int(N), int(M), ctypes.byref(out))
    return rc, (out.value if rc == CAST_OK else None)


def cast_plan_create_ex(tensors: Sequence[cast_tensor_t], N: int, M: int, plan_flags: int):
    """Returns (status, plan handle or None); plan_flags: OR of CAST_F_EMIT_COMPRESSED, CAST_F_MASK_STATS, or 0."""
    n = len(tensors)
    arr = (cast_tensor_t * max(n, 1))(*tensors)
    out = ctypes.c_void_p(None)
    rc = load_library().cast_plan_create_ex(arr if n else None, n, int(N), int(M), int(plan_flags), ctypes.byref(out))
    return rc, (out.value if rc == CAST_OK else None)


def make_hyper(lr, beta1, beta2, eps, l1_coeff, step, total_steps, flags) -> cast_hyper_t:
    return cast_hyper_t(lr, beta1, beta2, eps, l1_coeff, int(step), int(total_steps), int(flags))


def cast_plan_step(plan, hyper: Optional[cast_hyper_t], flip_count=None, stream=None) -> int:
    h = ctypes.byref(hyper) if hyper is not None else None
    return load_library().cast_plan_step(plan, h, _ptr(flip_count), _stream(stream))


def cast_plan_step_stats(plan, hyper: Optional[cast_hyper_t], flip_count=None, stats=None, stream=None) -> int:
    """`stats`: device buffer of sizeof(cast_mask_stats_t) = 32 bytes that a step with CAST_F_MASK_STATS adds to."""
    h = ctypes.byref(hyper) if hyper is not None else None
    return load_library().cast_plan_step_stats(plan, h, _ptr(flip_count), _ptr(stats), _stream(stream))


def cast_plan_report_staging_failure(plan) -> int:
    return load_library().cast_plan_report_staging_failure(plan)


def cast_plan_destroy(plan) -> int:
    return load_library().cast_plan_destroy(plan)


def cast_host_ctx_create(max_block_params: int, n_slots: int):
    """Returns (status, context handle or None)."""
    out = ctypes.c_void_p(None)
    rc = load_library().cast_host_ctx_create(int(max_block_params), int(n_slots), ctypes.byref(out))
    return rc, (out.value if rc == CAST_OK else None)


def cast_host_step(ctx, w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols, N, M,
                   lr, beta1, beta2, eps, l1_coeff, step, total_steps, flags, flip_count=None) -> int:
    return load_library().cast_host_step(
        ctx, _ptr(w), _ptr(m), _ptr(v), _ptr(g), _ptr(w_fwd_bf16), _ptr(meta), _ptr(scale), int(scale_groups),
        int(rows), int(cols), int(N), int(M), lr, beta1, beta2, eps, l1_coeff, int(step), int(total_steps),
        int(flags), _ptr(flip_count))


CAST_STATIC_MAX_PARAMS = 1048576


def cast_host_step_static(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols, N, M,
                          lr, beta1, beta2, eps, l1_coeff, step, total_steps, flags, flip_count=None, stream=None) -> int:
    """cast_host_step through the staging area built into the library: host pointers in and out, no device
    allocation by the call, at most CAST_STATIC_MAX_PARAMS parameters, synchronous on `stream`."""
    return load_library().cast_host_step_static(
        _ptr(w), _ptr(m), _ptr(v), _ptr(g), _ptr(w_fwd_bf16), _ptr(meta), _ptr(scale), int(scale_groups),
        int(rows), int(cols), int(N), int(M), lr, beta1, beta2, eps, l1_coeff, int(step), int(total_steps),
        int(flags), _ptr(flip_count), _stream(stream))


def cast_kd_loss(student_logits, teacher_logits, labels, loss, grad_logits, tokens, vocab, eta, grad_scale=1.0, stream=None) -> int:
    return load_library().cast_kd_loss(_ptr(student_logits), _ptr(teacher_logits), _ptr(labels), _ptr(loss), _ptr(grad_logits),
                                       int(tokens), int(vocab), eta, grad_scale, _stream(stream))


def cast_prune_fold(w, scale, scale_groups, meta, out, rows, cols, N, M, flags, stream=None) -> int:
    return load_library().cast_prune_fold(_ptr(w), _ptr(scale), int(scale_groups), _ptr(meta), _ptr(out), int(rows), int(cols),
                                          int(N), int(M), int(flags), _stream(stream))


def cast_plan_prune_fold(plan, outs, flags, stream=None) -> int:
    """`outs`: a sequence of one output buffer per matrix of the plan."""
    arr = None if outs is None else (ctypes.c_void_p * len(outs))(*[_ptr(o) for o in outs])
    return load_library().cast_plan_prune_fold(plan, arr, int(flags), _stream(stream))


class cast_mask_stats_t(ctypes.Structure):
    _fields_ = [("mask_diff", ctypes.c_ulonglong), ("reserved_", ctypes.c_ulonglong),
                ("kept_abs_sum", ctypes.c_double), ("total_abs_sum", ctypes.c_double)]


def cast_mask_stats(w, meta, meta_ref, rows, cols, M, flags, stats, stream=None) -> int:
    """`stats`: device buffer of sizeof(cast_mask_stats_t) = 32 bytes that the call adds to."""
    return load_library().cast_mask_stats(_ptr(w), _ptr(meta), _ptr(meta_ref), int(rows), int(cols), int(M), int(flags),
                                          _ptr(stats), _stream(stream))


def cast_plan_mask_stats(plan, meta_refs, flags, stats, stream=None) -> int:
    """`meta_refs`: a sequence of one reference-mask buffer per matrix of the plan, or None."""
    arr = None
    if meta_refs is not None:
        arr = (ctypes.c_void_p * len(meta_refs))(*[_ptr(r) for r in meta_refs])
    return load_library().cast_plan_mask_stats(plan, arr, int(flags), _ptr(stats), _stream(stream))


def cast_bulk_timeout_count():
    """Returns (status, count)."""
    out = ctypes.c_ulonglong(0)
    rc = load_library().cast_bulk_timeout_count(ctypes.byref(out))
    return rc, int(out.value)


def cast_probe_launch(n_ctas, stream=None) -> int:
    return load_library().cast_probe_launch(int(n_ctas), _stream(stream))


def cast_probe_stream(w, m, v, g, w_fwd, meta, n_params, stream=None) -> int:
    return load_library().cast_probe_stream(_ptr(w), _ptr(m), _ptr(v), _ptr(g), _ptr(w_fwd), _ptr(meta), int(n_params),
                                            _stream(stream))


def cast_host_ctx_sync(ctx) -> int:
    return load_library().cast_host_ctx_sync(ctx)


def cast_host_ctx_destroy(ctx) -> int:
    return load_library().cast_host_ctx_destroy(ctx)
