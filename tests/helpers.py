"""Small numpy helpers of the tests (decoding written independently of both implementations)."""
from __future__ import annotations

import numpy as np
import torch


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def torch_bf16_bits(x_f32: np.ndarray) -> np.ndarray:
    """bf16 bits of fp32 values by the library conversion (round to nearest even)."""
    t = torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def keep_mask_from_meta(meta: np.ndarray, cols: int, M: int, bitmask: bool) -> np.ndarray:
    """Boolean [rows, cols] keep mask decoded from the metadata words.

    A word describes 32 consecutive columns of a row, fields of M bits packed
    from the least significant bit.  bitmask=True: bit j of a field = column
    j of the group is kept.  bitmask=False (2:4 only): field = lo | hi << 2,
    the positions of the two kept columns."""
    meta = np.asarray(meta, dtype=np.uint32).reshape(-1, cols // 32)
    rows = meta.shape[0]
    bits = ((meta[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).astype(np.uint8)
    bits = bits.reshape(rows, cols)
    if bitmask:
        return bits.astype(bool)
    assert M == 4
    nib = bits.reshape(rows, cols // 4, 4)
    lo = nib[:, :, 0] + 2 * nib[:, :, 1]
    hi = nib[:, :, 2] + 2 * nib[:, :, 3]
    keep = np.zeros((rows, cols // 4, 4), dtype=bool)
    r, gidx = np.meshgrid(np.arange(rows), np.arange(cols // 4), indexing="ij")
    keep[r, gidx, lo] = True
    keep[r, gidx, hi] = True
    return keep.reshape(rows, cols)


def within_tol(got: np.ndarray, ref: np.ndarray, rel: float = 1e-6, floor: float = 1e-9):
    """|got - ref| <= max(rel * |ref|, floor) element-wise; returns (ok, worst excess ratio)."""
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    err = np.abs(got - ref)
    bound = np.maximum(rel * np.abs(ref), floor)
    ratio = err / bound
    return bool(np.all(ratio <= 1.0)), float(ratio.max() if ratio.size else 0.0)


def bf16_ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in bf16 units in the last place between two arrays of raw bf16 bits
    (sign-magnitude mapped onto a monotone integer line; +0 and -0 coincide)."""
    def key(b):
        b = b.astype(np.int32)
        mag = b & 0x7FFF
        return np.where(b & 0x8000, -mag, mag)
    return np.abs(key(a_bits) - key(b_bits))
