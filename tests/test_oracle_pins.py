"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's loop: each one compares it with a
brute-force enumeration, a value the paper prints, a closed form that holds at
special parameter values, or a library routine (torch.optim.Adam, torch's bf16
conversion).  They run without a GPU.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import adams_oracle as orc
from oracle.adams_oracle import Hyper
from helpers import bf16_bits_to_f32, keep_mask_from_meta, torch_bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

NM_CASES = [(1, 2), (1, 4), (2, 4), (3, 4), (4, 4), (4, 8), (2, 8), (1, 8), (5, 16), (8, 16)]


def zeros_like_state(rows, cols):
    z = np.zeros((rows, cols), dtype=np.float32)
    return z.copy(), z.copy(), np.zeros((rows, cols), dtype=np.uint16)


def run(w, m=None, v=None, g=None, scale=None, N=2, M=4, hyper=None, flags=orc.F_RESELECT | orc.F_META_BITMASK,
        meta_in=None, precision="f64"):
    rows, cols = w.shape
    zm, zv, zg = zeros_like_state(rows, cols)
    m = zm if m is None else m
    v = zv if v is None else v
    g = zg if g is None else g
    hyper = hyper or Hyper()
    return orc.adams_step(w, m, v, g, scale, N, M, hyper, flags, meta_in, precision)


def bf16_exact(x):
    """fp32 array whose values are exactly representable in bf16, and their bits."""
    bits = torch_bf16_bits(np.asarray(x, dtype=np.float32))
    return bf16_bits_to_f32(bits), bits


# --------------------------------------------------------------------------- selection (Eq. 3, 4, 6)

def adversarial_groups(rng, n_groups, M):
    w = rng.normal(0, 0.02, size=(n_groups, M)).astype(np.float32)
    # exact ties, equal magnitudes of opposite sign, zeros of both signs, all-equal groups
    w[0::7, 1 % M] = w[0::7, 0]
    w[1::7, M - 1] = -w[1::7, 0]
    w[2::7, :] = 0.0
    w[3::7, 0] = -0.0
    w[4::7, :] = 0.125
    w[5::7, M // 2] = 0.0
    return w


@pytest.mark.parametrize("N,M", NM_CASES)
def test_selection_is_the_brute_force_maximum(N, M):
    rng = np.random.default_rng(100 * N + M)
    n_groups = 32 * 12
    groups = adversarial_groups(rng, n_groups, M)
    cols = 64 if M <= 16 else 128
    w = groups.reshape(-1, cols)
    out = run(w, N=N, M=M, hyper=Hyper(lr=0.0))
    keep = keep_mask_from_meta(out["meta"], cols, M, bitmask=True).reshape(n_groups, M)
    a = np.abs(groups.astype(np.float64))
    combos = [np.array(c) for c in itertools.combinations(range(M), N)]
    for gi in range(n_groups):
        assert keep[gi].sum() == N                                        # Eq. 4
        sums = np.array([a[gi, c].sum() for c in combos])
        assert a[gi, keep[gi]].sum() == sums.max()                        # Eq. 6: the N largest magnitudes
        if len(np.unique(a[gi])) == M:                                    # no ties: the mask is unique
            assert set(np.flatnonzero(keep[gi])) == set(combos[int(sums.argmax())])
        else:                                                             # ties go to the lower column
            order = sorted(range(M), key=lambda j: (-a[gi, j], j))
            assert set(np.flatnonzero(keep[gi])) == set(order[:N])


def test_paper_one_two_example():
    rows = []
    with open(os.path.join(GOLDEN, "one_two_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            lhs, rhs = line.split("->")
            rows.append(([float(x) for x in lhs.split()], [float(x) for x in rhs.split()]))
    assert len(rows) == 2
    for theta, fwd in rows:
        w = np.tile(np.array(theta, dtype=np.float32), 16)[None, :]          # 32 columns: 16 copies of the pair
        out = run(w, N=1, M=2, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT | orc.F_META_BITMASK)
        got = bf16_bits_to_f32(out["w_fwd"])[0, :2]
        expect = bf16_bits_to_f32(torch_bf16_bits(np.array(fwd, dtype=np.float32)))
        assert np.array_equal(got, expect)
        keep = keep_mask_from_meta(out["meta"], 32, 2, True)[0, :2]
        assert list(keep) == [f != 0 for f in fwd]


@pytest.mark.parametrize("N,M", NM_CASES)
def test_every_group_keeps_exactly_n(N, M):
    rng = np.random.default_rng(7)
    w = rng.normal(0, 0.02, size=(5, 96 if M < 32 else 128)).astype(np.float32)
    cols = w.shape[1]
    if cols % M:
        pytest.skip("shape")
    out = run(w, N=N, M=M)
    keep = keep_mask_from_meta(out["meta"], cols, M, True)
    assert np.all(keep.reshape(5, cols // M, M).sum(-1) == N)
    assert out["meta"].nbytes == w.size // 8                                # one bit per parameter
    fwd = bf16_bits_to_f32(out["w_fwd"])
    assert np.all(fwd[~keep] == 0) and np.all(out["w_fwd"][~keep] == 0)      # pruned slots are +0


# --------------------------------------------------------------------------- Adam core

def torch_adam_reference(w0, grads, lr, beta1, beta2, eps):
    p = torch.nn.Parameter(torch.from_numpy(w0.astype(np.float64)))
    opt = torch.optim.Adam([p], lr=lr, betas=(beta1, beta2), eps=eps, weight_decay=0.0)
    for g in grads:
        p.grad = torch.from_numpy(g.astype(np.float64))
        opt.step()
    st = opt.state[p]
    return p.detach().numpy(), st["exp_avg"].numpy(), st["exp_avg_sq"].numpy()


@pytest.mark.parametrize("beta1,flags_extra", [(0.0, 0), (0.9, orc.F_V_KEPT_FROM_G)])
def test_reduces_to_textbook_adam(beta1, flags_extra):
    """l1_coeff = 0 and full density (N = M): the literal update equals Adam when beta1 = 0
    (v is fed by the first moment, Eq. 8); with kept entries feeding g^2 it equals Adam for any beta1."""
    rng = np.random.default_rng(3)
    rows, cols, steps = 6, 64, 6
    w0 = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    grads = [bf16_exact(rng.normal(0, 1e-3, size=(rows, cols)))[0] for _ in range(steps)]
    h = dict(lr=1e-3, beta1=beta1, beta2=0.95, eps=1e-8)
    hf = {k: float(np.float32(x)) for k, x in h.items()}
    ref_w, ref_m, ref_v = torch_adam_reference(w0, grads, hf["lr"], hf["beta1"], hf["beta2"], hf["eps"])
    w, m, v = w0.copy(), np.zeros_like(w0), np.zeros_like(w0)
    for t, g in enumerate(grads, start=1):
        out = run(w, m, v, torch_bf16_bits(g), N=4, M=4,
                  hyper=Hyper(l1_coeff=0.0, step=t, total_steps=1000, **h),
                  flags=orc.F_RESELECT | orc.F_META_BITMASK | flags_extra)
        w, m, v = out["w"], out["m"], out["v"]
    np.testing.assert_allclose(w, ref_w, rtol=2e-6, atol=1e-10)
    np.testing.assert_allclose(m, ref_m, rtol=2e-6, atol=5e-11)     # fp32 storage of m, cancellation
    np.testing.assert_allclose(v, ref_v, rtol=2e-6, atol=1e-18)


def test_literal_reading_differs_from_adam_when_beta1_nonzero():
    """Guard on the reading itself: with beta1 = 0.9 the literal second moment (from mu^2) is not Adam's."""
    rng = np.random.default_rng(4)
    w0 = rng.normal(0, 0.02, size=(2, 32)).astype(np.float32)
    g, gb = bf16_exact(rng.normal(0, 1e-3, size=(2, 32)))
    out = run(w0, g=gb, N=4, M=4, hyper=Hyper(l1_coeff=0.0, step=1, total_steps=10))
    _, _, ref_v = torch_adam_reference(w0, [g], 1e-4, float(np.float32(0.9)), float(np.float32(0.95)), 1e-8)
    assert np.all(out["v"] < 0.02 * ref_v + 1e-30)          # (1-beta1)^2 = 0.01 of g^2


def test_first_step_closed_form_kept_entry():
    """t = 1, m0 = v0 = 0, kept entry: dw = -lr g / ((1-beta1)|g| + eps); under the g^2 reading -lr g/(|g| + eps)."""
    g, gb = bf16_exact(np.array([[3e-3, -2e-3, 5e-4, -7e-5] * 8]))
    w0 = np.full((1, 32), 0.5, dtype=np.float32)
    h = Hyper(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, l1_coeff=0.3, step=1, total_steps=50)
    lr, b1, b2, eps, _ = h.as_f32()
    out = run(w0, g=gb, N=4, M=4, hyper=h)
    expect = 0.5 - lr * g.astype(np.float64) / ((1 - b1) * np.abs(g) + eps)
    np.testing.assert_allclose(out["w"], expect, rtol=1e-7)
    out2 = run(w0, g=gb, N=4, M=4, hyper=h, flags=orc.F_RESELECT | orc.F_META_BITMASK | orc.F_V_KEPT_FROM_G)
    expect2 = 0.5 - lr * g.astype(np.float64) / (np.abs(g) + eps)
    np.testing.assert_allclose(out2["w"], expect2, rtol=1e-7)


# --------------------------------------------------------------------------- proportional L1 decay (Eq. 7)

def group_with_known_mask(sign=1.0):
    """2:4 groups (4, 3, 2, 1) * 0.01 * sign: columns 0, 1 kept, columns 2, 3 masked."""
    return (np.tile(np.array([4, 3, 2, 1], dtype=np.float32), 8)[None, :] * np.float32(0.01) * np.float32(sign))


@pytest.mark.parametrize("sign", [1.0, -1.0])
def test_decay_closed_form_at_alpha_one(sign):
    """alpha = 1 (t = T), g = 0, m = 0, v0 = lambda^2, masked entry: mu~ = lambda Sign(w), v stays
    lambda^2, dw = -lr (lambda/bc1) Sign(w) / (lambda/sqrt(bc2) + eps); kept entries do not move."""
    w0 = group_with_known_mask(sign)
    lam = float(np.float32(2e-3))
    h = Hyper(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, l1_coeff=lam, step=20, total_steps=20)
    lr, b1, b2, eps, _ = h.as_f32()
    v0 = np.full_like(w0, np.float32(lam) ** 2)
    out = run(w0, v=v0, N=2, M=4, hyper=h)
    bc1, bc2 = 1 - b1 ** 20, 1 - b2 ** 20
    v_expect = b2 * float(v0[0, 0]) + (1 - b2) * lam * lam
    step_size = lr * (lam / bc1) / (np.sqrt(v_expect / bc2) + eps)
    masked = np.tile(np.array([False, False, True, True]), 8)[None, :]
    expect = w0.astype(np.float64) - np.where(masked, sign * step_size, 0.0)
    np.testing.assert_allclose(out["w"], expect, rtol=2e-7)
    np.testing.assert_allclose(out["v"][masked], v_expect, rtol=2e-7)
    np.testing.assert_allclose(out["v"][~masked], b2 * float(v0[0, 0]), rtol=2e-7)
    assert np.all(out["m"] == 0)                                   # the stored moment carries no decay


def test_decay_mixes_moment_and_sign_with_alpha():
    """t = 1 of T = 4 (alpha = 1/4), m0 = v0 = 0: mu = (1-b1) g, mu~ = 3/4 mu + 1/4 lambda Sign(w),
    v^ = mu~^2, so dw = -lr mu~ / ((1-b1)(|mu~| + eps... )) with the bias corrections of t = 1."""
    w0 = group_with_known_mask(1.0)
    g, gb = bf16_exact(np.full((1, 32), -6e-3))
    lam = float(np.float32(1e-3))
    h = Hyper(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, l1_coeff=lam, step=1, total_steps=4)
    lr, b1, b2, eps, _ = h.as_f32()
    out = run(w0, g=gb, N=2, M=4, hyper=h)
    mu = (1 - b1) * g.astype(np.float64)
    masked = np.tile(np.array([False, False, True, True]), 8)[None, :]
    mu_t = np.where(masked, 0.75 * mu + 0.25 * lam * 1.0, mu)
    expect_w = w0 - lr * (mu_t / (1 - b1)) / (np.abs(mu_t) + eps)
    np.testing.assert_allclose(out["w"], expect_w, rtol=2e-7)
    np.testing.assert_allclose(out["m"], mu, rtol=2e-7)            # stored first moment is undecayed
    np.testing.assert_allclose(out["v"], (1 - b2) * mu_t ** 2, rtol=3e-7)


def test_kept_entries_ignore_lambda_and_stored_moment_is_plain_ema():
    rng = np.random.default_rng(11)
    w0 = rng.normal(0, 0.02, size=(4, 64)).astype(np.float32)
    m0 = rng.normal(0, 1e-4, size=(4, 64)).astype(np.float32)
    v0 = (rng.normal(0, 1e-3, size=(4, 64)) ** 2).astype(np.float32)
    g, gb = bf16_exact(rng.normal(0, 1e-3, size=(4, 64)))
    a = run(w0, m0, v0, gb, N=2, M=4, hyper=Hyper(l1_coeff=0.0))
    b = run(w0, m0, v0, gb, N=2, M=4, hyper=Hyper(l1_coeff=0.5))
    keep = keep_mask_from_meta(a["meta"], 64, 4, True)
    assert np.array_equal(a["meta"], b["meta"])
    for k in ("w", "v", "w_fwd"):
        assert np.array_equal(a[k][keep], b[k][keep])
    assert not np.any(a["w"][~keep] == b["w"][~keep])
    assert np.array_equal(a["m"], b["m"])
    b1 = float(np.float32(0.9))
    ema = b1 * m0.astype(np.float64) + (1 - b1) * g.astype(np.float64)
    np.testing.assert_allclose(a["m"], ema, rtol=1e-6, atol=1e-12)


def test_alpha_to_zero_masked_path_meets_kept_path():
    rng = np.random.default_rng(12)
    w0 = rng.normal(0, 0.02, size=(4, 64)).astype(np.float32)
    m0 = rng.normal(0, 1e-4, size=(4, 64)).astype(np.float32)
    v0 = (rng.normal(0, 1e-3, size=(4, 64)) ** 2).astype(np.float32)
    _, gb = bf16_exact(rng.normal(0, 1e-3, size=(4, 64)))
    h = Hyper(l1_coeff=1e-3, step=1, total_steps=10 ** 15)
    sparse = run(w0, m0, v0, gb, N=2, M=4, hyper=h)
    dense = run(w0, m0, v0, gb, N=4, M=4, hyper=h)
    np.testing.assert_allclose(sparse["w"], dense["w"], rtol=2e-7, atol=1e-12)
    np.testing.assert_allclose(sparse["v"], dense["v"], rtol=2e-7, atol=1e-20)


def test_sign_of_zero_is_zero_and_sign_follows_the_weight_immediately():
    w0 = group_with_known_mask(1.0)
    w0[0, 2] = 0.0          # masked (smallest magnitudes of its group are columns 2, 3)
    w0[0, 6] = -0.0
    rng = np.random.default_rng(13)
    m0 = rng.normal(0, 1e-4, size=w0.shape).astype(np.float32)
    v0 = np.full_like(w0, 1e-6)
    h = Hyper(l1_coeff=0.05, step=10, total_steps=20)
    with_decay = run(w0, m0, v0, N=2, M=4, hyper=h)
    # at a zero weight the decay term vanishes: same as lambda = 0
    no_lambda = run(w0, m0, v0, N=2, M=4, hyper=Hyper(l1_coeff=0.0, step=10, total_steps=20))
    for c in (2, 6):
        assert with_decay["w"][0, c] == no_lambda["w"][0, c]
        assert with_decay["v"][0, c] == no_lambda["v"][0, c]
    assert with_decay["w"][0, 3] != no_lambda["w"][0, 3]
    # the decay direction is read from the current weight, not from accumulated momentum:
    # a masked weight just below zero is pushed up although its neighbour just above zero is pushed down
    w1 = group_with_known_mask(1.0)
    w1[0, 2], w1[0, 3] = 1e-5, -1e-5
    out = run(w1, v=v0, N=2, M=4, hyper=Hyper(lr=1e-6, l1_coeff=0.05, step=20, total_steps=20))
    assert out["w"][0, 2] < w1[0, 2] and out["w"][0, 3] > w1[0, 3]
    assert np.isclose(w1[0, 2] - out["w"][0, 2], out["w"][0, 3] - w1[0, 3], rtol=1e-3)


# --------------------------------------------------------------------------- weight scaling, emission (Eq. 11, 12)

def edge_floats():
    rng = np.random.default_rng(21)
    vals = [0.0, -0.0, 1.0, -1.0, 1.00390625, 1.01171875, 1.005859375, 1.0058593, 1.0058594,   # ties and near ties
            3.3895314e38, 3.4e38, 1e-38, 1e-40, 9.1835e-41, 4.5e-41, 1e-45, 65504.0, 0.1, -0.3, 255.5, 256.5, 257.5]
    x = np.array(vals, dtype=np.float32)
    # every bf16 mid-point pattern: low 16 bits = 0x8000 (tie), 0x7FFF, 0x8001 around random upper halves
    hi = rng.integers(0x0000, 0x7F00, size=600, dtype=np.uint32) << 16
    lows = np.array([0x8000, 0x7FFF, 0x8001, 0x0000, 0xFFFF, 0x0001], dtype=np.uint32)
    bits = (hi[:, None] | lows[None, :]).reshape(-1)
    sign = (rng.integers(0, 2, size=bits.size, dtype=np.uint32) << 31)
    y = (bits | sign).astype(np.uint32).view(np.float32)
    z = rng.normal(0, 1, size=2000).astype(np.float32) * np.float32(10.0) ** rng.integers(-30, 30, size=2000).astype(np.float32)
    allv = np.concatenate([x, y, z.astype(np.float32)])
    pad = (-allv.size) % 32
    return np.concatenate([allv, np.ones(pad, dtype=np.float32)])[None, :]


@pytest.mark.parametrize("precision", ["f64", "f32"])
def test_bf16_rounding_matches_library_conversion(precision):
    w0 = edge_floats()
    out = run(w0, N=4, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT | orc.F_META_BITMASK | orc.F_EMIT_DENSE,
              precision=precision)
    assert np.array_equal(out["w"].view(np.uint32), w0.view(np.uint32))       # lr = 0 leaves w untouched
    assert np.array_equal(out["w_fwd"], torch_bf16_bits(w0))


def test_unit_scale_emits_masked_bf16_of_updated_weight_and_pow2_scale_is_exact():
    rng = np.random.default_rng(22)
    rows, cols = 6, 128
    w0 = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    m0 = rng.normal(0, 1e-4, size=(rows, cols)).astype(np.float32)
    v0 = (rng.normal(0, 1e-3, size=(rows, cols)) ** 2).astype(np.float32)
    _, gb = bf16_exact(rng.normal(0, 1e-3, size=(rows, cols)))
    none = run(w0, m0, v0, gb, scale=None)
    ones = run(w0, m0, v0, gb, scale=np.ones((rows, 2), dtype=np.float32))
    keep = keep_mask_from_meta(none["meta"], cols, 4, True)
    expect = np.where(keep, torch_bf16_bits(none["w"]), np.uint16(0))
    assert np.array_equal(none["w_fwd"], expect) and np.array_equal(ones["w_fwd"], expect)
    for k in (3, -2):
        sc = np.full((rows, 2), 2.0 ** k, dtype=np.float32)
        out = run(w0, m0, v0, gb, scale=sc)
        assert np.array_equal(out["w"], none["w"])                           # the optimizer acts on raw W
        assert np.array_equal(bf16_bits_to_f32(out["w_fwd"]), bf16_bits_to_f32(expect) * np.float32(2.0 ** k))


@pytest.mark.parametrize("n_seg", [1, 2, 4])
def test_scale_segment_of_a_column(n_seg):
    """Eq. 12: row r is cut into n contiguous segments of C/n columns; segment s uses A[r, s]."""
    rows, cols = 3, 128
    w0 = np.full((rows, cols), 0.5, dtype=np.float32)
    scale = (2.0 ** (np.arange(rows)[:, None] * 4 + np.arange(n_seg)[None, :])).astype(np.float32)
    out = run(w0, scale=scale, N=4, M=4, hyper=Hyper(lr=0.0))
    got = bf16_bits_to_f32(out["w_fwd"])
    for r in range(rows):
        for c in range(cols):
            assert got[r, c] == 0.5 * scale[r, c // (cols // n_seg)]


def test_dense_emission_keeps_masked_entries():
    w0 = group_with_known_mask(1.0)
    out = run(w0, N=2, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT | orc.F_META_BITMASK | orc.F_EMIT_DENSE)
    assert np.array_equal(out["w_fwd"], torch_bf16_bits(w0))


# --------------------------------------------------------------------------- metadata, mask reuse, flips

def test_index_and_bitmask_encodings_describe_the_same_mask():
    rng = np.random.default_rng(31)
    w0 = rng.normal(0, 0.02, size=(7, 96)).astype(np.float32)
    a = run(w0, N=2, M=4, flags=orc.F_RESELECT | orc.F_META_BITMASK, hyper=Hyper(lr=0.0))
    b = run(w0, N=2, M=4, flags=orc.F_RESELECT, hyper=Hyper(lr=0.0))
    nonzero = bf16_bits_to_f32(a["w_fwd"]) != 0        # weights are nonzero, so kept <=> emitted nonzero
    assert np.array_equal(keep_mask_from_meta(a["meta"], 96, 4, True), nonzero)
    assert np.array_equal(keep_mask_from_meta(b["meta"], 96, 4, False), nonzero)
    nibbles = (b["meta"][:, :, None] >> (4 * np.arange(8, dtype=np.uint32))[None, None, :]) & 0xF
    assert np.all((nibbles & 3) < (nibbles >> 2))                          # lower position first
    assert a["meta"].nbytes == b["meta"].nbytes == w0.size // 8


def test_hand_packed_word_layout():
    """One row of 64 columns, 2:4: keep columns {1,2} in group 0, {0,3} in group 8, {2,3} in group 15."""
    w0 = np.tile(np.array([4, 3, 2, 1], dtype=np.float32), 16)[None, :].copy()     # default: keep {0,1}
    w0[0, 0:4] = [1, 4, 3, 2]
    w0[0, 32:36] = [4, 1, 2, 3]
    w0[0, 60:64] = [1, 2, 3, 4]
    bm = run(w0, N=2, M=4, hyper=Hyper(lr=0.0))["meta"]
    ix = run(w0, N=2, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT)["meta"]
    word0_bm = sum(0b0011 << (4 * k) for k in range(1, 8)) | 0b0110
    word1_bm = sum(0b0011 << (4 * k) for k in range(1, 7)) | 0b1001 | (0b1100 << 28)
    idx = lambda lo, hi: lo | (hi << 2)
    word0_ix = sum(idx(0, 1) << (4 * k) for k in range(1, 8)) | idx(1, 2)
    word1_ix = sum(idx(0, 1) << (4 * k) for k in range(1, 7)) | idx(0, 3) | (idx(2, 3) << 28)
    assert [int(x) for x in bm[0]] == [word0_bm, word1_bm]
    assert [int(x) for x in ix[0]] == [word0_ix, word1_ix]


@pytest.mark.parametrize("bitmask", [True, False])
def test_reused_mask_is_decoded_and_flips_are_counted(bitmask):
    enc = orc.F_META_BITMASK if bitmask else 0
    rng = np.random.default_rng(32)
    w0 = rng.normal(0, 0.02, size=(4, 64)).astype(np.float32)
    first = run(w0, N=2, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT | enc)
    # same weights again: no flips
    again = run(w0, N=2, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT | orc.F_COUNT_FLIPS | enc, meta_in=first["meta"])
    assert again["flips"] == 0 and np.array_equal(again["meta"], first["meta"])
    # a hand-made previous mask: every group keeps {0, 1}
    field = 0b0011 if bitmask else (0 | 1 << 2)
    prev = np.full((4, 2), sum(field << (4 * k) for k in range(8)), dtype=np.uint32)
    keep = keep_mask_from_meta(first["meta"], 64, 4, bitmask)
    hand = int(np.sum(keep != np.tile(np.array([True, True, False, False]), 16)[None, :]))
    cnt = run(w0, N=2, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT | orc.F_COUNT_FLIPS | enc, meta_in=prev)
    assert cnt["flips"] == hand and hand > 0
    # mask reuse (no reselection): the given mask gates decay and emission even though it is not the top-2
    reuse = run(w0, N=2, M=4, hyper=Hyper(lr=0.0), flags=enc, meta_in=prev)
    assert np.array_equal(reuse["meta"], prev)
    assert np.array_equal(bf16_bits_to_f32(reuse["w_fwd"]) != 0, np.tile(np.array([True, True, False, False]), 16)[None, :].repeat(4, 0))


@pytest.mark.parametrize("bitmask", [True, False])
def test_stored_mask_gates_the_decay_when_it_is_not_the_top_n(bitmask):
    """Mask reuse (no reselection) with a stored mask that is NOT the magnitude top-2: every group of
    (4, 3, 2, 1) * 0.01 stores the kept set {2, 3}, the two SMALLEST entries.  With alpha = 1, g = 0, m = 0,
    v0 = lambda^2 the closed form of Eq. 7 says exactly which entries move: the ones outside the STORED set
    (columns 0, 1) shrink by lr (lambda/bc1) / (lambda/sqrt(bc2) + eps) and feed lambda^2 into v; the stored
    kept entries (columns 2, 3) do not move and their v only decays.  Had the decay been gated by a freshly
    selected set (columns 0, 1 kept) the roles would be swapped."""
    enc = orc.F_META_BITMASK if bitmask else 0
    w0 = group_with_known_mask(1.0)
    lam = float(np.float32(2e-3))
    h = Hyper(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, l1_coeff=lam, step=20, total_steps=20)
    lr, b1, b2, eps, _ = h.as_f32()
    v0 = np.full_like(w0, np.float32(lam) ** 2)
    field = 0b1100 if bitmask else (2 | 3 << 2)
    stored = np.full((1, 1), sum(field << (4 * k) for k in range(8)), dtype=np.uint32)
    out = run(w0, v=v0, N=2, M=4, hyper=h, flags=enc, meta_in=stored)
    bc1, bc2 = 1 - b1 ** 20, 1 - b2 ** 20
    v_decayed = b2 * float(v0[0, 0])
    v_masked = v_decayed + (1 - b2) * lam * lam
    step_size = lr * (lam / bc1) / (np.sqrt(v_masked / bc2) + eps)
    outside = np.tile(np.array([True, True, False, False]), 8)[None, :]          # outside the stored set
    np.testing.assert_allclose(out["w"], w0.astype(np.float64) - np.where(outside, step_size, 0.0), rtol=2e-7)
    assert np.array_equal(out["w"][~outside], w0[~outside])
    np.testing.assert_allclose(out["v"][outside], v_masked, rtol=2e-7)
    np.testing.assert_allclose(out["v"][~outside], v_decayed, rtol=2e-7)
    assert np.array_equal(out["meta"], stored)                                   # a reused mask is left as it is
    assert np.array_equal(bf16_bits_to_f32(out["w_fwd"]) != 0, ~outside)         # and it prunes the emitted weight
    # the freshly selected set on the same inputs moves the other half
    fresh = run(w0, v=v0, N=2, M=4, hyper=h, flags=orc.F_RESELECT | enc)
    assert np.array_equal(fresh["w"][outside], w0[outside]) and not np.any(fresh["w"][~outside] == w0[~outside])


def test_chain_rule_factor_is_the_scale_passed_to_the_call():
    """With the gradient taken through the scaling (Eq. 12) the oracle multiplies g by the scale it is given in THIS
    call -- also when that scale differs from the one an earlier call emitted the forward weight with (the one-step
    lag the header describes).  beta1 = 0, t = 1, m0 = v0 = 0, full density: the stored first moment is exactly
    A (.) g, per row segment, for whatever A is passed; the emitted weight uses the same A."""
    rng = np.random.default_rng(77)
    w0 = rng.normal(0, 0.02, size=(3, 64)).astype(np.float32)
    g, gb = bf16_exact(rng.normal(0, 1e-3, size=(3, 64)))
    a_old = (1 + 0.1 * rng.random((3, 2))).astype(np.float32)
    a_new = (a_old * np.float32(1.25)).astype(np.float32)                  # an exact, visible change of the scale
    h = Hyper(lr=1e-4, beta1=0.0, beta2=0.95, eps=1e-8, l1_coeff=0.0, step=1, total_steps=10)
    flags = orc.F_RESELECT | orc.F_META_BITMASK | orc.F_GRAD_OF_SCALED | orc.F_EMIT_DENSE
    for a in (a_old, a_new):
        out = run(w0, g=gb, scale=a, N=4, M=4, hyper=h, flags=flags)
        seg = np.repeat(a, 32, axis=1).astype(np.float64)
        np.testing.assert_allclose(out["m"], seg * g, rtol=1e-7)
        np.testing.assert_allclose(bf16_bits_to_f32(out["w_fwd"]), seg * out["w"], rtol=2.0 ** -8)
        np.testing.assert_allclose(out["scale_grad"], (g.astype(np.float64) * w0).reshape(3, 2, 32).sum(-1), rtol=1e-12)
    # the exact form: the forward pass used A_old (chain-rule factor), this step emits with A_new.  torch autograd
    # on L = sum(c (.) (A_old (.) W)) gives dL/dW = A_old (.) c: that is what the stored first moment must be.
    W = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
    A_f = torch.tensor(np.repeat(a_old, 32, axis=1), dtype=torch.float64)
    (torch.tensor(g, dtype=torch.float64) * (A_f * W)).sum().backward()
    out = orc.adams_step(w0, np.zeros_like(w0), np.zeros_like(w0), gb, a_new, 4, 4, h, flags, scale_chain=a_old)
    np.testing.assert_allclose(out["m"], W.grad.numpy(), rtol=1e-7)
    np.testing.assert_allclose(bf16_bits_to_f32(out["w_fwd"]), np.repeat(a_new, 32, axis=1) * out["w"].astype(np.float64), rtol=2.0 ** -8)
    both = orc.adams_step(w0, np.zeros_like(w0), np.zeros_like(w0), gb, a_old, 4, 4, h, flags)
    assert np.array_equal(out["m"], both["m"]) and np.array_equal(out["w"], both["w"])      # only the emission differs


# --------------------------------------------------------------------------- numerics and long-run behaviour

def test_fp32_order_stays_within_tolerance_of_fp64():
    rng = np.random.default_rng(41)
    rows, cols = 16, 256
    w0 = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    m0 = rng.normal(0, 1e-4, size=(rows, cols)).astype(np.float32)
    v0 = (rng.normal(0, 1e-3, size=(rows, cols)) ** 2).astype(np.float32)
    _, gb = bf16_exact(rng.normal(0, 1e-3, size=(rows, cols)))
    sc = (1 + 0.1 * rng.random((rows, 2))).astype(np.float32)
    a = run(w0, m0, v0, gb, scale=sc, precision="f64")
    b = run(w0, m0, v0, gb, scale=sc, precision="f32")
    assert np.array_equal(a["meta"], b["meta"])
    for k in ("w", "m", "v"):
        err = np.abs(a[k].astype(np.float64) - b[k]) / np.maximum(1e-6 * np.abs(a[k]), 1e-9)
        assert err.max() < 0.5, (k, err.max())
    da = bf16_bits_to_f32(a["w_fwd"]).astype(np.float64)
    db = bf16_bits_to_f32(b["w_fwd"])
    assert np.all(np.abs(da - db) <= np.abs(da) * 2.0 ** -7)


def _refresh_schedule_worst_excess(lr):
    """Steps t = 9, 10, 11 of a T = 12 run (mask refreshed and flips counted at t = 10, reused otherwise) on the
    16 x 2048 seeded inputs of the GPU refresh-schedule test: worst |f32 - f64| / max(1e-6 |f64|, 1e-9) of w
    over the three steps, each step of both builds starting from the fp64 build's previous state."""
    from paper_2509_25996_b200 import workloads
    from helpers import within_tol
    rows, cols = 16, 2048
    inp = workloads.gen_tensor_inputs(rows, cols, seed=9, tensor_index=0, device="cpu", scale_mode="jitter")
    w, m, v, sc = inp.w.numpy(), inp.m.numpy(), inp.v.numpy(), inp.scale.numpy()
    meta = orc.adams_step(w, m, v, workloads.bf16_bits(inp.g), sc, 2, 4, Hyper(lr=0.0), orc.F_RESELECT)["meta"]
    worst = 0.0
    for t in (9, 10, 11):
        flags = (orc.F_RESELECT | orc.F_COUNT_FLIPS) if t % 10 == 0 else 0
        h = Hyper(lr=lr, l1_coeff=1e-3, step=t, total_steps=12)
        gb = workloads.bf16_bits(workloads.gen_gradient(rows, cols, 9, 0, t))
        a = orc.adams_step(w, m, v, gb, sc, 2, 4, h, flags, meta, "f64")
        b = orc.adams_step(w, m, v, gb, sc, 2, 4, h, flags, meta, "f32")
        assert np.array_equal(a["meta"], b["meta"])
        for k in ("m", "v"):
            assert within_tol(b[k], a[k])[0]
        worst = max(worst, within_tol(b["w"], a["w"])[1])
        w, m, v, meta = a["w"], a["m"], a["v"], a["meta"]
    return worst


def test_accuracy_domain_of_fp32_evaluation():
    """The accepted error max(1e-6 |w|, 1e-9) has an absolute floor, so it bounds the per-step update for which
    ANY fp32 evaluation of Alg. 1 can meet it: the update lr mu^/(sqrt(v^) + eps) carries a relative rounding
    error of a few 2^-24, i.e. the floor is reached once the update is a few 1e-3.  With beta = 0.9 / 0.95 the
    ratio mu^/sqrt(v^) is at most ~4.5, so lr = 5e-3 gives updates up to ~2e-2 and lr = 2e-4 up to ~1e-3.
    The fp32 build of the oracle (plain IEEE operations in the written order) leaves the tolerance at the
    first and stays well inside it at the second: the domain in which the tolerance is meaningful for an
    fp32 implementation is per-step updates below ~1e-3, which every listed workload (lr = 1e-4) satisfies."""
    assert _refresh_schedule_worst_excess(5e-3) > 1.5
    assert _refresh_schedule_worst_excess(2e-4) < 0.5


def test_masked_weights_shrink_as_alpha_ramps():
    """Smoke test of the long-run behaviour the paper describes (App. C: the kept share of the
    magnitude tends to 1); exact trajectories are not printed anywhere, so nothing is compared."""
    rng = np.random.default_rng(42)
    rows, cols, T = 8, 64, 300
    w = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    m = np.zeros_like(w)
    v = np.zeros_like(w)
    meta = None
    ratios = []
    for t in range(1, T + 1):
        _, gb = bf16_exact(rng.normal(0, 1e-4, size=(rows, cols)))
        flags = orc.F_META_BITMASK | (orc.F_RESELECT if (t == 1 or t % 10 == 0) else 0)
        out = run(w, m, v, gb, hyper=Hyper(lr=2e-3, l1_coeff=1e-4, step=t, total_steps=T), flags=flags, meta_in=meta)
        w, m, v, meta = out["w"], out["m"], out["v"], out["meta"]
        keep = keep_mask_from_meta(meta, cols, 4, True)
        ratios.append(np.abs(w[keep]).sum() / np.abs(w).sum())
    assert ratios[-1] > 0.97 and ratios[-1] > ratios[0] + 0.1


# --------------------------------------------------------------------------- mask statistics (App. C)

@pytest.mark.parametrize("N,M,bitmask", [(2, 4, False), (2, 4, True), (4, 8, True), (1, 4, True), (5, 16, True)])
def test_mask_statistics_match_numpy_on_an_independently_decoded_mask(N, M, bitmask):
    rng = np.random.default_rng(50 + M)
    rows, cols = 7, 192
    enc = orc.F_META_BITMASK if bitmask else 0
    w = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    w_ref = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    meta = run(w, N=N, M=M, flags=orc.F_RESELECT | enc)["meta"]
    meta_ref = run(w_ref, N=N, M=M, flags=orc.F_RESELECT | enc)["meta"]
    w_now = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)     # statistics take any W with any mask
    got = orc.mask_stats(w_now, meta, meta_ref, M, bitmask)
    keep = keep_mask_from_meta(meta, cols, M, bitmask)
    keep_ref = keep_mask_from_meta(meta_ref, cols, M, bitmask)
    a = np.abs(w_now.astype(np.float64))
    assert got["flips"] == int(np.sum(keep != keep_ref)) > 0
    assert got["kept_abs"] == pytest.approx(float(a[keep].sum()), rel=1e-13)
    assert got["total_abs"] == pytest.approx(float(a.sum()), rel=1e-13)
    assert orc.mask_stats(w_now, meta, None, M, bitmask)["flips"] == 0


def test_mask_statistics_closed_forms():
    rng = np.random.default_rng(60)
    rows, cols = 3, 64
    w = rng.normal(0, 1, size=(rows, cols)).astype(np.float32)
    # full density: every entry kept, S_t = 1; a mask against itself: no flips
    full = run(w, N=4, M=4)["meta"]
    s = orc.mask_stats(w, full, full, 4, True)
    assert s["flips"] == 0 and s["kept_abs"] == s["total_abs"] > 0
    # complementary 2:4 masks (keep {0, 1} against keep {2, 3}) differ in every entry
    lo = np.full((rows, cols // 32), 0x33333333, dtype=np.uint32)
    hi = np.full((rows, cols // 32), 0xCCCCCCCC, dtype=np.uint32)
    assert orc.mask_stats(w, lo, hi, 4, True)["flips"] == rows * cols
    # the same two masks in index form: nibble 0x4 = positions (0, 1), nibble 0xE = positions (2, 3)
    lo_i = np.full((rows, cols // 32), 0x44444444, dtype=np.uint32)
    hi_i = np.full((rows, cols // 32), 0xEEEEEEEE, dtype=np.uint32)
    si = orc.mask_stats(w, lo_i, hi_i, 4, False)
    assert si["flips"] == rows * cols
    assert si["kept_abs"] == pytest.approx(float(np.abs(w.astype(np.float64)).reshape(-1, 4)[:, :2].sum()), rel=1e-13)
    # a hand-sized case: one row of 32 columns, keep columns 0 and 3 of every group; |w| = 1, 2, 3, 4 repeating
    w1 = np.tile(np.array([1, -2, 3, -4], dtype=np.float32), 8)[None, :]
    m1 = np.full((1, 1), 0x99999999, dtype=np.uint32)
    s1 = orc.mask_stats(w1, m1, None, 4, True)
    assert s1["kept_abs"] == 8 * (1 + 4) and s1["total_abs"] == 8 * 10


def test_sparse_weight_ratio_rises_as_alpha_ramps():
    """App. C: with the decay ramping up, masked magnitudes shrink and S_t moves toward 1 (smoke test)."""
    rng = np.random.default_rng(61)
    rows, cols = 8, 128
    w = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    m = np.zeros_like(w)
    v = np.full_like(w, 1e-6)
    g = np.zeros((rows, cols), dtype=np.uint16)
    ratios = []
    T = 60
    for t in range(1, T + 1):
        out = run(w, m, v, g, N=2, M=4, hyper=Hyper(lr=1e-3, l1_coeff=1e-3, step=t, total_steps=T))
        w, m, v = out["w"], out["m"], out["v"]
        s = orc.mask_stats(w, out["meta"], None, 4, True)
        ratios.append(s["kept_abs"] / s["total_abs"])
    assert ratios[-1] > ratios[0] and ratios[-1] > 0.9


# --------------------------------------------------------------------------- compressed emission (Alg. 2, final loop)

@pytest.mark.parametrize("N,M,bitmask", [(2, 4, False), (2, 4, True), (1, 4, True), (3, 4, True), (4, 8, True), (1, 2, True), (5, 16, True)])
def test_compressed_emission_is_the_pruned_matrix_without_its_pruned_slots(N, M, bitmask):
    """The compressed forward weight holds, group by group and in column order, exactly the entries the pruned
    form keeps: gathering the pruned form through an independently decoded mask gives it, and scattering it
    back through that mask gives the pruned form."""
    rng = np.random.default_rng(70 + M + N)
    rows, cols = 5, 160
    w = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    g = bf16_exact(rng.normal(0, 1e-3, size=(rows, cols)))[1]
    scale = (1.0 + 0.1 * rng.random((rows, 2))).astype(np.float32)
    enc = orc.F_META_BITMASK if bitmask else 0
    dense = run(w, g=g, scale=scale, N=N, M=M, flags=orc.F_RESELECT | enc)
    comp = run(w, g=g, scale=scale, N=N, M=M, flags=orc.F_RESELECT | enc | orc.F_EMIT_COMPRESSED)
    for k in ("w", "m", "v", "meta"):
        assert np.array_equal(dense[k], comp[k])
    assert comp["w_fwd"].shape == (rows, cols * N // M)
    keep = keep_mask_from_meta(dense["meta"], cols, M, bitmask)
    assert np.array_equal(comp["w_fwd"].reshape(-1), dense["w_fwd"][keep])        # row-major gather keeps column order
    back = np.zeros((rows, cols), dtype=np.uint16)
    back[keep] = comp["w_fwd"].reshape(-1)
    assert np.array_equal(back, dense["w_fwd"])


def test_compressed_emission_hand_example():
    """One row, 2:4, weights that do not move (lr = 0), scale 2: the kept pair of every group, doubled."""
    w = np.tile(np.array([0.5, -4.0, 3.0, 0.25, 1.0, 1.0, -1.0, 0.125], dtype=np.float32), 4)[None, :]
    out = run(w, N=2, M=4, scale=np.full((1, 2), 2.0, dtype=np.float32), hyper=Hyper(lr=0.0),
              flags=orc.F_RESELECT | orc.F_EMIT_COMPRESSED)
    want = np.tile(np.array([-8.0, 6.0, 2.0, 2.0], dtype=np.float32), 4)            # ties: the lower columns (1.0, 1.0)
    assert np.array_equal(bf16_bits_to_f32(out["w_fwd"]).reshape(-1), want)


# --------------------------------------------------------------------------- gradient through the scaling (Eq. 12)

@pytest.mark.parametrize("n_seg", [1, 2, 4])
def test_gradient_of_the_scaled_weight_follows_autograd(n_seg):
    """With g the gradient of the loss with respect to W_scale = Diag(A) W, the chain rule is checked against
    torch autograd on the linear loss <W_scale, g>: dL/dA is the oracle's scale gradient, and dL/dW is what the
    first moment sees (m_0 = 0, so m_1 = (1 - beta1) dL/dW)."""
    rng = np.random.default_rng(80 + n_seg)
    rows, cols = 6, 128
    w = rng.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    g32, g_bits = bf16_exact(rng.normal(0, 1e-3, size=(rows, cols)))
    scale = (1.0 + 0.5 * rng.random((rows, n_seg))).astype(np.float32)
    A = torch.tensor(scale, dtype=torch.float64, requires_grad=True)
    W = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    loss = ((A.repeat_interleave(cols // n_seg, dim=1) * W) * torch.tensor(g32, dtype=torch.float64)).sum()
    loss.backward()
    h = Hyper(beta1=0.9)
    out = run(w, g=g_bits, scale=scale, N=2, M=4, hyper=h, flags=orc.F_RESELECT | orc.F_META_BITMASK | orc.F_GRAD_OF_SCALED)
    assert np.allclose(out["scale_grad"], A.grad.numpy(), rtol=1e-12, atol=0)
    b1 = float(np.float32(0.9))
    assert np.allclose(out["m"], ((1.0 - b1) * W.grad.numpy()).astype(np.float32), rtol=1e-6, atol=0)
    # without the flag the same g is taken as dL/dW itself, and no scale gradient is produced
    plain = run(w, g=g_bits, scale=scale, N=2, M=4, hyper=h)
    assert plain["scale_grad"] is None
    assert np.allclose(plain["m"], ((1.0 - b1) * g32).astype(np.float32), rtol=1e-6, atol=0)
    # a unit scale makes the two readings coincide
    ones = np.ones((rows, n_seg), dtype=np.float32)
    a = run(w, g=g_bits, scale=ones, N=2, M=4, hyper=h, flags=orc.F_RESELECT | orc.F_META_BITMASK | orc.F_GRAD_OF_SCALED)
    b = run(w, g=g_bits, scale=ones, N=2, M=4, hyper=h)
    for k in ("w", "m", "v", "w_fwd", "meta"):
        assert np.array_equal(a[k], b[k])


def test_plain_adam_for_the_scale_matches_torch():
    rng = np.random.default_rng(90)
    theta0 = (1.0 + 0.1 * rng.random(64)).astype(np.float32)
    theta, m, v = theta0.copy(), np.zeros(64, np.float32), np.zeros(64, np.float32)
    p = torch.tensor(theta0.astype(np.float64), requires_grad=True)
    opt = torch.optim.Adam([p], lr=1e-3, betas=(float(np.float32(0.9)), float(np.float32(0.95))), eps=float(np.float32(1e-8)))
    for t in range(1, 6):
        grad = rng.normal(0, 1e-2, size=64).astype(np.float32)
        theta, m, v = orc.plain_adam(theta, m, v, grad, float(np.float32(1e-3)), 0.9, 0.95, 1e-8, t)
        p.grad = torch.tensor(grad.astype(np.float64))
        opt.step()
        # the oracle stores fp32 state between steps, torch keeps fp64: a few fp32 roundings per step
        assert np.allclose(theta, p.detach().numpy(), rtol=5e-7 * t, atol=0)


# --------------------------------------------------------------------------- final pruning (Alg. 2, final loop)

@pytest.mark.parametrize("N,M,bitmask", [(2, 4, False), (2, 4, True), (1, 4, True), (4, 8, True), (3, 4, True), (5, 16, True), (8, 32, True)])
def test_final_pruning_against_stable_argsort_and_library_bf16(N, M, bitmask):
    """Kept set by numpy's stable sort of -|w| (equal magnitudes keep column order), values by torch's bf16
    conversion of the fp32 product, the two output layouts by gather/scatter through the decoded mask."""
    rng = np.random.default_rng(100 + M + N)
    rows, cols = 6, 192
    w = adversarial_groups(rng, rows * cols // M, M).reshape(rows, cols)
    scale = np.ldexp(1.0, rng.integers(-2, 3, size=(rows, 2))).astype(np.float32)      # powers of two: a*w is exact in fp32
    enc = orc.F_META_BITMASK if bitmask else 0
    dense = orc.prune_fold(w, scale, N, M, orc.F_RESELECT | enc)
    order = np.argsort(-np.abs(w.reshape(-1, M)), axis=1, kind="stable")[:, :N]
    want_keep = np.zeros((rows * cols // M, M), dtype=bool)
    np.put_along_axis(want_keep, order, True, axis=1)
    want_keep = want_keep.reshape(rows, cols)
    assert np.array_equal(keep_mask_from_meta(dense["meta"], cols, M, bitmask), want_keep)
    a_full = np.repeat(scale, cols // 2, axis=1)
    want = np.where(want_keep, torch_bf16_bits(a_full * w), 0).astype(np.uint16)
    assert np.array_equal(dense["out"], want)
    comp = orc.prune_fold(w, scale, N, M, orc.F_RESELECT | enc | orc.F_EMIT_COMPRESSED)
    assert np.array_equal(comp["meta"], dense["meta"])
    assert np.array_equal(comp["out"].reshape(-1), want[want_keep])
    # a stored mask is used as it is, whatever the weights are now
    other = rng.normal(0, 1, size=(rows, cols)).astype(np.float32)
    reuse = orc.prune_fold(other, None, N, M, enc, meta_in=dense["meta"])
    assert np.array_equal(reuse["meta"], dense["meta"])
    assert np.array_equal(reuse["out"], np.where(want_keep, torch_bf16_bits(other), 0).astype(np.uint16))


def test_final_pruning_is_the_step_emission_of_unmoved_weights():
    """Consistency of the two oracles: with a zero learning rate the AdamS step leaves W alone, and its emitted
    forward weight is the final pruning of W."""
    rng = np.random.default_rng(110)
    w = rng.normal(0, 0.02, size=(4, 128)).astype(np.float32)
    scale = (1.0 + 0.1 * rng.random((4, 2))).astype(np.float32)
    step = run(w, scale=scale, N=2, M=4, hyper=Hyper(lr=0.0), flags=orc.F_RESELECT)
    pf = orc.prune_fold(w, scale, 2, 4, orc.F_RESELECT)
    assert np.array_equal(step["w_fwd"], pf["out"]) and np.array_equal(step["meta"], pf["meta"])


# --------------------------------------------------------------------------- distillation loss (Eq. 13)

def _logits(rng, tokens, vocab, spread):
    x = torch.tensor(rng.normal(0, spread, size=(tokens, vocab)), dtype=torch.float32).to(torch.bfloat16)
    return x, x.view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("eta", [0.0, 1.0 / 3.0, 1.0])
def test_distillation_loss_and_gradient_follow_torch(eta):
    rng = np.random.default_rng(120)
    tokens, vocab = 5, 257
    s, s_bits = _logits(rng, tokens, vocab, 3.0)
    t, t_bits = _logits(rng, tokens, vocab, 4.0)
    labels = np.array([3, 256, 0, -100, 17], dtype=np.int32)
    eta32 = float(np.float32(eta))
    loss, grad = orc.kd_loss(s_bits, t_bits, labels, eta, grad_scale=0.25)
    S = s.to(torch.float64).requires_grad_(True)
    T = t.to(torch.float64)
    log_ps = torch.log_softmax(S, dim=-1)
    kl = torch.nn.functional.kl_div(log_ps, torch.softmax(T, dim=-1), reduction="none").sum(-1)
    ce = torch.nn.functional.cross_entropy(S, torch.tensor(labels, dtype=torch.long), ignore_index=-100, reduction="none")
    want = eta32 * kl + (1.0 - eta32) * ce
    assert np.allclose(loss, want.detach().numpy(), rtol=1e-12, atol=1e-13)
    (float(np.float32(0.25)) * want.sum()).backward()
    assert np.allclose(grad, S.grad.numpy(), rtol=1e-10, atol=1e-15)


def test_distillation_loss_closed_forms():
    rng = np.random.default_rng(121)
    s, s_bits = _logits(rng, 3, 64, 2.0)
    labels = np.array([1, 2, 3], dtype=np.int32)
    # teacher == student: the KL term vanishes, and so does its gradient
    loss, grad = orc.kd_loss(s_bits, s_bits, labels, 1.0)
    assert np.all(np.abs(loss) < 1e-15) and np.all(np.abs(grad) < 1e-15)
    # a uniform student: cross-entropy is log V whatever the label; gradient 1/V - onehot
    zeros = np.zeros((3, 64), dtype=np.uint16)
    loss, grad = orc.kd_loss(zeros, s_bits, labels, 0.0)
    assert np.allclose(loss, np.log(64.0), rtol=1e-15)
    want = np.full((3, 64), 1.0 / 64)
    want[np.arange(3), labels] -= 1.0
    assert np.allclose(grad, want, rtol=1e-13, atol=1e-16)
    # gradients of a token sum to zero when it has a target (probabilities sum to one on both sides)
    loss, grad = orc.kd_loss(s_bits, _logits(rng, 3, 64, 2.0)[1], labels, 1.0 / 3.0)
    assert np.all(np.abs(grad.sum(-1)) < 1e-14)
