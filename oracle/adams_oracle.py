"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs
may import this module.  It takes and returns numpy arrays; it never touches a
GPU and never imports the CUDA package.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np

from . import build_oracle

# Flag values of the oracle (see adams_oracle.c).
F_RESELECT = 1
F_COUNT_FLIPS = 2
F_META_BITMASK = 4
F_V_KEPT_FROM_G = 8
F_EMIT_DENSE = 16
F_EMIT_COMPRESSED = 32
F_GRAD_OF_SCALED = 64

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_oracle.build())
        for name in ("oracle_adams_step_f64", "oracle_adams_step_f32"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [
                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,   # w m v g
                ctypes.c_void_p, ctypes.c_void_p,                                     # w_fwd meta
                ctypes.c_void_p, ctypes.c_int,                                        # scale n_seg
                ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,           # rows cols N M
                ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                ctypes.c_int64, ctypes.c_int64,                                       # step total_steps
                ctypes.c_uint32, ctypes.c_void_p,                                     # flags flip_count
                ctypes.c_void_p,                                                      # scale_grad
                ctypes.c_void_p,                                                      # scale_chain
            ]
        lib.oracle_prune_fold.restype = ctypes.c_int
        lib.oracle_prune_fold.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_uint32]
        lib.oracle_kd_loss.restype = ctypes.c_int
        lib.oracle_kd_loss.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                       ctypes.c_double, ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_plain_adam.restype = ctypes.c_int
        lib.oracle_plain_adam.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                          ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int64]
        lib.oracle_mask_stats.restype = ctypes.c_int
        lib.oracle_mask_stats.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                          ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


@dataclass
class Hyper:
    """Hyper-parameters of one step.  Values are rounded to fp32 first, because
    the CUDA entry points take them as fp32: both sides then see the same numbers."""
    lr: float = 1e-4
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    l1_coeff: float = 1e-3
    step: int = 1000
    total_steps: int = 30000

    def as_f32(self):
        f = lambda x: float(np.float32(x))
        return f(self.lr), f(self.beta1), f(self.beta2), f(self.eps), f(self.l1_coeff)


def adams_step_inplace(w, m, v, g_bits, w_fwd_bits, meta, scale, rows, cols, N, M, hyper: Hyper,
                       flags: int, precision: str = "f64", scale_grad=None, scale_chain=None) -> int:
    """Run the oracle in place on C-contiguous numpy arrays.

    w, m, v: float32 [rows*cols]; g_bits, w_fwd_bits: uint16 (raw bf16);
    meta: uint32 [rows*cols/32]; scale: float32 [rows, n_seg] or None.
    Returns the number of mask flips counted (0 unless F_COUNT_FLIPS)."""
    lib = _load()
    fn = lib.oracle_adams_step_f64 if precision == "f64" else lib.oracle_adams_step_f32
    for a, dt in ((w, np.float32), (m, np.float32), (v, np.float32), (g_bits, np.uint16),
                  (w_fwd_bits, np.uint16), (meta, np.uint32)):
        assert a.dtype == dt and a.flags["C_CONTIGUOUS"], (a.dtype, dt)
    assert w.size == rows * cols and meta.size == rows * cols // 32
    assert w_fwd_bits.size == (rows * cols * N // M if flags & F_EMIT_COMPRESSED else rows * cols)
    n_seg = 1
    scale_ptr = None
    if scale is not None:
        assert scale.dtype == np.float32 and scale.flags["C_CONTIGUOUS"] and scale.shape[0] == rows
        n_seg = scale.shape[1]
        scale_ptr = scale.ctypes.data
    if scale_grad is not None:
        assert scale_grad.dtype == np.float64 and scale_grad.flags["C_CONTIGUOUS"] and scale_grad.size == rows * n_seg
    chain_ptr = None
    if scale_chain is not None:
        assert scale is not None and scale_chain.dtype == np.float32 and scale_chain.flags["C_CONTIGUOUS"] and scale_chain.shape == scale.shape
        chain_ptr = scale_chain.ctypes.data
    flips = ctypes.c_uint64(0)
    lr, b1, b2, eps, lam = hyper.as_f32()
    rc = fn(w.ctypes.data, m.ctypes.data, v.ctypes.data, g_bits.ctypes.data,
            w_fwd_bits.ctypes.data, meta.ctypes.data, scale_ptr, n_seg,
            rows, cols, N, M, lr, b1, b2, eps, lam, hyper.step, hyper.total_steps,
            flags, ctypes.addressof(flips), None if scale_grad is None else scale_grad.ctypes.data, chain_ptr)
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (status {rc})")
    return int(flips.value)


def adams_step(w, m, v, g_bits, scale, N, M, hyper: Hyper, flags: int = F_RESELECT,
               meta_in=None, precision: str = "f64", scale_chain=None):
    """Out-of-place convenience wrapper for 2-D inputs.

    Returns dict(w, m, v, w_fwd (uint16 bf16 bits; [rows, cols*N/M] with F_EMIT_COMPRESSED), meta (uint32
    [rows, cols/32]), flips)."""
    rows, cols = w.shape
    w2 = np.ascontiguousarray(w, dtype=np.float32).copy().reshape(-1)
    m2 = np.ascontiguousarray(m, dtype=np.float32).copy().reshape(-1)
    v2 = np.ascontiguousarray(v, dtype=np.float32).copy().reshape(-1)
    g2 = np.ascontiguousarray(g_bits, dtype=np.uint16).reshape(-1)
    fwd_cols = cols * N // M if flags & F_EMIT_COMPRESSED else cols
    fwd = np.zeros(rows * fwd_cols, dtype=np.uint16)
    if meta_in is None:
        meta = np.zeros(rows * cols // 32, dtype=np.uint32)
    else:
        meta = np.ascontiguousarray(meta_in, dtype=np.uint32).copy().reshape(-1)
    sc = None if scale is None else np.ascontiguousarray(scale, dtype=np.float32)
    scale_grad = None
    if flags & F_GRAD_OF_SCALED:
        scale_grad = np.zeros((rows, 1 if sc is None else sc.shape[1]), dtype=np.float64)
    chain = None if scale_chain is None else np.ascontiguousarray(scale_chain, dtype=np.float32)
    flips = adams_step_inplace(w2, m2, v2, g2, fwd, meta, sc, rows, cols, N, M, hyper, flags, precision, scale_grad, chain)
    return dict(scale_grad=scale_grad, w=w2.reshape(rows, cols), m=m2.reshape(rows, cols), v=v2.reshape(rows, cols),
                w_fwd=fwd.reshape(rows, fwd_cols), meta=meta.reshape(rows, cols // 32), flips=flips)


def mask_stats(w, meta, meta_ref, M: int, bitmask: bool):
    """Mask statistics of App. C for one matrix: dict(flips = ||M - M_ref||_0 (0 without meta_ref),
    kept_abs = ||W (.) M||_1, total_abs = ||W||_1), sums in fp64.  w: float32 [rows, cols]; meta, meta_ref:
    uint32 [rows, cols/32]."""
    lib = _load()
    rows, cols = w.shape
    w = np.ascontiguousarray(w, dtype=np.float32)
    meta = np.ascontiguousarray(meta, dtype=np.uint32)
    assert meta.size == rows * cols // 32
    ref_ptr = None
    if meta_ref is not None:
        meta_ref = np.ascontiguousarray(meta_ref, dtype=np.uint32)
        assert meta_ref.size == meta.size
        ref_ptr = meta_ref.ctypes.data
    flips = ctypes.c_uint64(0)
    sums = (ctypes.c_double * 2)(0.0, 0.0)
    rc = lib.oracle_mask_stats(w.ctypes.data, meta.ctypes.data, ref_ptr, rows, cols, M, 1 if bitmask else 0,
                               ctypes.addressof(flips), ctypes.addressof(sums))
    if rc != 0:
        raise ValueError("oracle_mask_stats rejected its arguments")
    return dict(flips=int(flips.value), kept_abs=float(sums[0]), total_abs=float(sums[1]))


def plain_adam(theta, m, v, grad, lr, beta1, beta2, eps, step):
    """Textbook Adam with bias correction on float32 arrays (copies returned): the optimizer of the scale matrix."""
    lib = _load()
    t2, m2, v2 = (np.ascontiguousarray(a, dtype=np.float32).copy() for a in (theta, m, v))
    g2 = np.ascontiguousarray(grad, dtype=np.float32)
    f = lambda x: float(np.float32(x))
    rc = lib.oracle_plain_adam(t2.ctypes.data, m2.ctypes.data, v2.ctypes.data, g2.ctypes.data, t2.size,
                               f(lr), f(beta1), f(beta2), f(eps), int(step))
    if rc != 0:
        raise ValueError("oracle_plain_adam rejected its arguments")
    return t2, m2, v2


def prune_fold(w, scale, N, M, flags: int = F_RESELECT, meta_in=None):
    """Final pruning with the scale folded in (Alg. 2, final loop).  flags: F_RESELECT, F_META_BITMASK,
    F_EMIT_COMPRESSED.  Returns dict(out (uint16 bf16 bits, [rows, cols] or [rows, cols*N/M]), meta)."""
    lib = _load()
    rows, cols = w.shape
    w = np.ascontiguousarray(w, dtype=np.float32)
    meta = np.zeros(rows * cols // 32, dtype=np.uint32) if meta_in is None else \
        np.ascontiguousarray(meta_in, dtype=np.uint32).copy().reshape(-1)
    ocols = cols * N // M if flags & F_EMIT_COMPRESSED else cols
    out = np.zeros(rows * ocols, dtype=np.uint16)
    sc = None if scale is None else np.ascontiguousarray(scale, dtype=np.float32)
    rc = lib.oracle_prune_fold(w.ctypes.data, None if sc is None else sc.ctypes.data, 1 if sc is None else sc.shape[1],
                               meta.ctypes.data, out.ctypes.data, rows, cols, N, M, flags)
    if rc != 0:
        raise ValueError("oracle_prune_fold rejected its arguments")
    return dict(out=out.reshape(rows, ocols), meta=meta.reshape(rows, cols // 32))


def kd_loss(student_bits, teacher_bits, labels, eta: float, grad_scale: float = 1.0, want_grad: bool = True):
    """Per-token loss of Eq. 13 and its gradient with respect to the student logits (both fp64).
    student_bits, teacher_bits: uint16 (raw bf16) [tokens, vocab]; labels: int32 [tokens] (negative: no target)."""
    lib = _load()
    s = np.ascontiguousarray(student_bits, dtype=np.uint16)
    t = np.ascontiguousarray(teacher_bits, dtype=np.uint16)
    y = np.ascontiguousarray(labels, dtype=np.int32)
    tokens, vocab = s.shape
    assert t.shape == s.shape and y.shape == (tokens,)
    loss = np.zeros(tokens, dtype=np.float64)
    grad = np.zeros((tokens, vocab), dtype=np.float64) if want_grad else None
    rc = lib.oracle_kd_loss(s.ctypes.data, t.ctypes.data, y.ctypes.data, tokens, vocab, float(np.float32(eta)),
                            float(np.float32(grad_scale)), loss.ctypes.data, None if grad is None else grad.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_kd_loss rejected its arguments")
    return loss, grad
