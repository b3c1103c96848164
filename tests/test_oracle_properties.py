"""Structural invariants of the CPU oracle that the mathematics of Alg. 1 fixes, whatever its arithmetic does:
rows and groups are independent problems (Eq. 3), the kept set depends on magnitudes only and is unchanged by a
positive power-of-two factor (Eq. 6), the flip count is the population count of the difference of the two decoded
masks (App. C), and bitmask and index metadata lead to the same numbers."""
import numpy as np
import pytest

from oracle import adams_oracle as orc
from oracle.adams_oracle import Hyper
from helpers import keep_mask_from_meta

RS, BM, FL = orc.F_RESELECT, orc.F_META_BITMASK, orc.F_COUNT_FLIPS


def state(rows, cols, seed):
    rng = np.random.default_rng(seed)
    w = rng.normal(0, 0.02, (rows, cols)).astype(np.float32)
    m = rng.normal(0, 1e-4, (rows, cols)).astype(np.float32)
    v = (rng.normal(0, 1e-3, (rows, cols)) ** 2).astype(np.float32)
    g = (rng.normal(0, 1e-3, (rows, cols)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    return w, m, v, g


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8), (1, 4), (5, 16)])
def test_rows_are_independent_problems(N, M):
    rows, cols = 6, 64
    w, m, v, g = state(rows, cols, 1)
    h = Hyper(l1_coeff=1e-3, step=1000, total_steps=7500)
    whole = orc.adams_step(w, m, v, g, None, N, M, h, RS | BM)
    perm = np.array([3, 0, 5, 1, 4, 2])
    shuffled = orc.adams_step(w[perm], m[perm], v[perm], g[perm], None, N, M, h, RS | BM)
    for k in ("w", "m", "v", "w_fwd", "meta"):
        assert np.array_equal(whole[k][perm], shuffled[k]), k
    for r in range(rows):
        one = orc.adams_step(w[r:r + 1], m[r:r + 1], v[r:r + 1], g[r:r + 1], None, N, M, h, RS | BM)
        for k in ("w", "m", "v", "w_fwd", "meta"):
            assert np.array_equal(whole[k][r:r + 1], one[k]), (k, r)


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8), (8, 32)])
def test_a_group_sees_only_its_own_columns(N, M):
    rows, cols = 3, 96
    w, m, v, g = state(rows, cols, 2)
    h = Hyper(l1_coeff=1e-3, step=500, total_steps=7500)
    base = orc.adams_step(w, m, v, g, None, N, M, h, RS | BM)
    w2 = w.copy()
    lo = (cols // M // 2) * M                       # one group in the middle of row 1 gets other weights
    w2[1, lo:lo + M] = np.linspace(0.5, 1.0, M, dtype=np.float32)
    other = orc.adams_step(w2, m, v, g, None, N, M, h, RS | BM)
    untouched = np.ones((rows, cols), dtype=bool)
    untouched[1, lo:lo + M] = False
    for k in ("w", "m", "v", "w_fwd"):
        assert np.array_equal(base[k][untouched], other[k][untouched]), k
    keep_a = keep_mask_from_meta(base["meta"], cols, M, True)
    keep_b = keep_mask_from_meta(other["meta"], cols, M, True)
    assert np.array_equal(keep_a[untouched], keep_b[untouched])
    assert np.array_equal(base["m"], other["m"])    # the stored first moment never depends on the weights


@pytest.mark.parametrize("N,M", [(2, 4), (1, 4), (4, 8), (8, 16)])
def test_kept_set_depends_on_magnitudes_only(N, M):
    rows, cols = 4, 64
    w, m, v, g = state(rows, cols, 3)
    h = Hyper(lr=0.0)
    ref = keep_mask_from_meta(orc.adams_step(w, m, v, g, None, N, M, h, RS | BM)["meta"], cols, M, True)
    for variant in (-w, np.abs(w), w * np.float32(8.0), w * np.float32(0.125)):
        got = keep_mask_from_meta(orc.adams_step(variant.astype(np.float32), m, v, g, None, N, M, h, RS | BM)["meta"], cols, M, True)
        assert np.array_equal(ref, got)
    assert np.all(ref.reshape(rows, cols // M, M).sum(-1) == N)


def test_flip_count_is_the_difference_of_the_decoded_masks_in_both_encodings():
    rows, cols = 5, 128
    w, m, v, g = state(rows, cols, 4)
    w_prev, _, _, _ = state(rows, cols, 5)
    h = Hyper(l1_coeff=1e-3, step=10, total_steps=100)
    for enc, bitmask in ((0, False), (BM, True)):
        prev = orc.adams_step(w_prev, m, v, g, None, 2, 4, Hyper(lr=0.0), RS | enc)["meta"]
        out = orc.adams_step(w, m, v, g, None, 2, 4, h, RS | FL | enc, meta_in=prev)
        a = keep_mask_from_meta(prev, cols, 4, bitmask)
        b = keep_mask_from_meta(out["meta"], cols, 4, bitmask)
        assert out["flips"] == int(np.count_nonzero(a != b)) > 0
        if bitmask:
            by_bitmask = out
        else:
            by_index = out
    for k in ("w", "m", "v", "w_fwd"):
        assert np.array_equal(by_index[k], by_bitmask[k]), k
    assert by_index["flips"] == by_bitmask["flips"]
