"""Pins for the oracle's arithmetic: constants, the AdamW inverse, the BF16 cast
and the changed set.  None of these compare the oracle with itself: they use
exact rational arithmetic, hand-worked cases, a forward AdamW step, an fp64
nearest-neighbour cast, a library cast and an unfused numpy evaluation."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from synth.tensors import Hyper, Spec, forward_adamw, make_state

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                yield line.split()


def f32_from_bits(b):
    return np.array([b], dtype=np.uint32).view(np.float32)[0]


def bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def fraction_to_f32_via_double(fr: Fraction) -> np.float32:
    # Fraction -> nearest double (Python's conversion is correctly rounded) -> fp32
    return np.float32(float(fr))


# ---------------------------------------------------------------- constants

def test_constants_match_golden_bit_patterns():
    got = {}
    for t in (1, 100, 500):
        c = bits(oracle.derive_constants(t, 1e-6, 0.9, 0.999, 1e-8, 0.01))
        got[("bc1", f"t={t}")] = c[0]
        got[("bc2", f"t={t}")] = c[1]
    for lr in (1e-6, 1e-4):
        for wd in (0.01, 0.1):
            c = bits(oracle.derive_constants(100, lr, 0.9, 0.999, 1e-8, wd))
            got[("decay", f"lr={lr:g},wd={wd:g}".replace("1e-06", "1e-6").replace("0.0001", "1e-4"))] = c[2]
    c = bits(oracle.derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.01))
    got[("lr", "lr=1e-6")] = c[3]
    got[("eps", "eps=1e-8")] = c[4]
    n = 0
    for name, arg, pat in _rows("constants.txt"):
        assert got[(name, arg)] == int(pat, 16), (name, arg, hex(got[(name, arg)]), pat)
        n += 1
    assert n == 12


@pytest.mark.parametrize("step", [1, 2, 3, 10, 100, 165, 500, 5000])
@pytest.mark.parametrize("b1,b2", [(0.9, 0.999), (0.5, 0.5), (0.95, 0.98)])
def test_constants_against_exact_rationals(step, b1, b2):
    lr, wd, eps = 3e-5, 0.1, 1e-8
    c = oracle.derive_constants(step, lr, b1, b2, eps, wd)
    exact = [1 - Fraction(b1) ** step, 1 - Fraction(b2) ** step, 1 - Fraction(lr) * Fraction(wd)]
    for got, fr in zip(c[:3], exact):
        want = fraction_to_f32_via_double(fr)
        # libm pow may be off by an ulp of double; after rounding to fp32 that can move the
        # result by at most one fp32 ulp, and only next to a rounding boundary.
        assert abs(int(bits(got)) - int(bits(want))) <= 1
        assert abs(Fraction(float(got)) - fr) <= Fraction(float(np.spacing(np.float32(want))))
    assert c[3] == np.float32(lr) and c[4] == np.float32(eps)


def test_decay_is_one_below_2_pow_minus_25():
    # 1 - lr*wd rounds to 1.0f as soon as lr*wd < 2^-25: weight decay then has no effect.
    assert oracle.derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.01)[2] == np.float32(1.0)
    assert oracle.derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.1)[2] < np.float32(1.0)


# ---------------------------------------------------------------- inverse: hand cases

def test_inverse_hand_cases():
    n = 0
    for rid, tb, mb, vb, lr, wd, eps, prev_b, bt, bp, changed in _rows("inverse_hand_cases.txt"):
        c = oracle.derive_constants(1, float(lr), 0.5, 0.5, float(eps), float(wd))
        assert c[0] == 0.5 and c[1] == 0.5
        th = np.array([int(tb, 16)], np.uint32).view(np.float32)
        m = np.array([int(mb, 16)], np.uint32).view(np.float32)
        v = np.array([int(vb, 16)], np.uint32).view(np.float32)
        prev = oracle.invert(th, m, v, c)
        assert bits(prev)[0] == int(prev_b, 16), rid
        assert oracle.bf16_rne(th)[0] == int(bt, 16), rid
        assert oracle.bf16_rne(prev)[0] == int(bp, 16), rid
        mask, val = oracle.changed_mask(th, m, v, c)
        assert int(mask[0]) == int(changed), rid
        assert val[0] == int(bt, 16), rid
        n += 1
    assert n == 8


# ---------------------------------------------------------------- inverse: forward step recovered

def _ulp_of_max(*arrs):
    M = np.maximum.reduce([np.abs(a.astype(np.float64)) for a in arrs])
    M = np.maximum(M, np.finfo(np.float32).tiny)
    return np.spacing(M.astype(np.float32)).astype(np.float64)


@pytest.mark.parametrize("variant,bound", [("mirror", 2.0), ("trainer", 4.0)])
@pytest.mark.parametrize("lr", [1e-8, 1e-6, 1e-4])
@pytest.mark.parametrize("step", [1, 100, 500])
@pytest.mark.parametrize("wd", [0.0, 0.01, 0.1])
def test_inverse_recovers_forward_step(variant, bound, lr, step, wd):
    hp = Hyper(step=step, lr=lr, wd=wd)
    st = make_state("w", 1 << 18, Spec(), hp, 7, "cpu", variant, keep_prev_fp32=True)
    theta, m, v, prev_true = (st[k].numpy() for k in ("theta", "m", "v", "prev"))
    c = oracle.derive_constants(*hp.as_args())
    prev = oracle.invert(theta, m, v, c)
    # |lr*u| from an fp64 evaluation of the update term
    u = (m.astype(np.float64) / c[0]) / (np.sqrt(v.astype(np.float64) / c[1]) + c[4])
    ulp = _ulp_of_max(prev_true, theta, (lr * u))
    err = np.abs(prev.astype(np.float64) - prev_true.astype(np.float64)) / ulp
    assert err.max() <= bound, err.max()
    if variant == "mirror":
        assert (prev == prev_true).mean() > 0.99


def test_inverse_matches_fp64_formula():
    # Eq. 2 evaluated in fp64 with the same fp32 constants: the fp32 procedure must stay
    # within a few ulp of the larger of |theta| and |lr*u|.  A dropped term, a sign flip, eps
    # inside the root or a swapped moment fails this by orders of magnitude.
    rng = np.random.default_rng(3)
    n = 200000
    theta = (rng.standard_normal(n) * 0.02).astype(np.float32)
    m = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    v = np.abs(rng.standard_normal(n) * 1e-5).astype(np.float32)
    v[:1000] = np.abs(rng.standard_normal(1000) * 1e-16).astype(np.float32)  # eps matters here
    for (step, lr, wd) in [(1, 1e-3, 0.1), (100, 1e-4, 0.01), (500, 1e-2, 0.5)]:
        c = oracle.derive_constants(step, lr, 0.9, 0.999, 1e-8, wd).astype(np.float64)
        t64, m64, v64 = (a.astype(np.float64) for a in (theta, m, v))
        upd = c[3] * (m64 / c[0]) / (np.sqrt(v64 / c[1]) + c[4])
        want = (t64 + upd) / c[2]
        got = oracle.invert(theta, m, v, c.astype(np.float32)).astype(np.float64)
        ulp = _ulp_of_max(want, theta, upd)
        assert (np.abs(got - want) / ulp).max() <= 4.0


def test_inverse_special_values():
    c = oracle.derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.01)
    sub = f32_from_bits(0x00000003)
    # m = v = 0: the update term is +0 and theta survives bit for bit, subnormals too
    # (except -0, which -0 + +0 = +0 turns into +0: hand case F)
    th = np.array([sub, -sub, 1.5, 0.0, 3e38], np.float32)
    z = np.zeros_like(th)
    assert np.array_equal(bits(oracle.invert(th, z, z, c)), bits(th))
    # v = 0, m != 0, eps > 0: finite, update = lr * (m/bc1)/eps
    got = oracle.invert(np.float32([1.0]), np.float32([1e-12]), np.float32([0.0]), c)
    want = 1.0 + float(c[3]) * (1e-12 / float(c[0])) / float(c[4])
    assert abs(got[0] - want) <= np.spacing(np.float32(1.0))
    # eps = 0 and m = v = 0 gives 0/0 = NaN; v < 0 gives NaN
    c0 = oracle.derive_constants(100, 1e-6, 0.9, 0.999, 0.0, 0.01)
    assert np.isnan(oracle.invert(np.float32([1.0]), np.float32([0.0]), np.float32([0.0]), c0)[0])
    assert np.isnan(oracle.invert(np.float32([1.0]), np.float32([1.0]), np.float32([-1.0]), c)[0])
    # Inf propagates
    assert np.isinf(oracle.invert(np.float32([np.inf]), np.float32([1.0]), np.float32([1.0]), c)[0])


# ---------------------------------------------------------------- BF16 cast

def _bf16_nearest_fp64(x32: np.ndarray) -> np.ndarray:
    """Nearest of the two neighbouring BF16 values, distances in fp64, ties to even."""
    u = x32.view(np.uint32).astype(np.uint64)
    lo = (u & 0xFFFF0000)
    hi = lo + 0x10000  # next BF16 away from zero (may be +-Inf; never wraps for finite x)
    lo_f = lo.astype(np.uint32).view(np.float32).astype(np.float64)
    hi_u32 = hi.astype(np.uint32)
    hi_f = hi_u32.view(np.float32).astype(np.float64)
    # beyond the largest finite BF16 the upper neighbour is 2^128 for rounding purposes
    is_inf = (hi_u32 & 0x7FFFFFFF) == 0x7F800000
    sign = np.where((u >> 31) == 1, -1.0, 1.0)
    hi_f = np.where(is_inf, sign * 2.0 ** 128, hi_f)
    x = x32.astype(np.float64)
    dlo, dhi = np.abs(x - lo_f), np.abs(hi_f - x)
    lo_even = ((lo >> 16) & 1) == 0
    pick_hi = (dhi < dlo) | ((dhi == dlo) & ~lo_even)
    return np.where(pick_hi, hi >> 16, lo >> 16).astype(np.uint16)


def _cast_inputs():
    rng = np.random.default_rng(11)
    hi = np.arange(1 << 16, dtype=np.uint32) << 16
    lows = np.array([0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x4000, 0xC000], np.uint32)
    grid = (hi[:, None] | lows[None, :]).reshape(-1)
    rnd = rng.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32)
    return np.concatenate([grid, rnd])


def test_bf16_rne_against_fp64_nearest_and_library_cast():
    u = _cast_inputs()
    x = u.view(np.float32)
    got = oracle.bf16_rne(x)
    finite_or_inf = ~np.isnan(x)
    want = _bf16_nearest_fp64(x[finite_or_inf])
    assert np.array_equal(got[finite_or_inf], want)
    # library cast (round-to-nearest-even) on everything that is not NaN
    lib = torch.from_numpy(x[finite_or_inf].copy()).to(torch.bfloat16).view(torch.int16).numpy()
    assert np.array_equal(got[finite_or_inf].view(np.int16), lib)
    # NaN of any sign / payload becomes the quiet pattern 0x7FC0
    assert np.all(got[~finite_or_inf] == 0x7FC0)
    assert (~finite_or_inf).sum() > 1000


def test_bf16_rne_every_fp32_pattern_against_the_library_cast():
    """All 2^32 inputs: the oracle's integer round-to-nearest-even equals torch's fp32 -> bf16 cast
    on every pattern that is not a NaN, and gives 0x7FC0 on every NaN."""
    import torch
    chunk = 1 << 20          # small enough for the allocator to reuse its buffers
    base = np.arange(chunk, dtype=np.uint32)
    nans = 0
    for lo in range(0, 1 << 32, chunk):
        bits = base + np.uint32(lo)
        got = oracle.bf16_rne(bits.view(np.float32))
        lib = torch.from_numpy(bits.view(np.int32)).view(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        nan = (bits & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
        if nan.any():
            assert np.all(got[nan] == 0x7FC0), hex(lo)
            assert np.array_equal(got[~nan], lib[~nan]), hex(lo)
            nans += int(nan.sum())
        else:
            assert np.array_equal(got, lib), hex(lo)
    assert nans == 2 * ((1 << 23) - 1)


def test_bf16_rne_named_cases():
    cases = {0x3F808000: 0x3F80, 0x3F818000: 0x3F82, 0x3F808001: 0x3F81, 0x3F807FFF: 0x3F80,
             0x7F7F8000: 0x7F80, 0x7F7F7FFF: 0x7F7F, 0xFF7F8000: 0xFF80, 0x00000000: 0x0000,
             0x80000000: 0x8000, 0x00008000: 0x0000, 0x00008001: 0x0001, 0x00018000: 0x0002,
             0x477FE000: 0x4780, 0x7F800000: 0x7F80, 0x7FC00000: 0x7FC0, 0xFFFFFFFF: 0x7FC0,
             0x7F800001: 0x7FC0}
    x = np.array(list(cases.keys()), np.uint32).view(np.float32)
    assert list(oracle.bf16_rne(x)) == list(cases.values())


# ---------------------------------------------------------------- changed set (Eq. 4), unfused

def _unfused_numpy(theta, m, v, c):
    """Array-at-a-time fp32 evaluation (numpy rounds every operation on its own)."""
    f = np.float32
    with np.errstate(all="ignore"):
        mhat = theta.dtype.type(0) + m / f(c[0])
        vhat = v / f(c[1])
        den = np.sqrt(vhat) + f(c[4])
        u = mhat / den
        prev = (theta + f(c[3]) * u) / f(c[2])
    assert prev.dtype == np.float32
    bt = _bf16_nearest_fp64(theta)
    bp = _bf16_nearest_fp64(prev)
    nan_t, nan_p = np.isnan(theta), np.isnan(prev)
    bt = np.where(nan_t, 0x7FC0, bt).astype(np.uint16)
    bp = np.where(nan_p, 0x7FC0, bp).astype(np.uint16)
    return prev, bt, bp


@pytest.mark.parametrize("lr,step,wd", [(1e-6, 100, 0.01), (1e-4, 1, 0.1), (1e-5, 500, 0.01),
                                        (1e-8, 100, 0.1)])
def test_changed_set_against_unfused_arrays(lr, step, wd):
    hp = Hyper(step=step, lr=lr, wd=wd)
    st = make_state("w", 300007, Spec(sigma_g=1e-2), hp, 5, "cpu")
    theta, m, v = (st[k].numpy() for k in ("theta", "m", "v"))
    theta = theta.copy()
    theta[::1001] = f32_from_bits(0x3F808000)
    theta[1::1001] = -0.0
    c = oracle.derive_constants(*hp.as_args())
    prev, bt, bp = _unfused_numpy(theta, m, v, c)
    assert np.array_equal(bits(oracle.invert(theta, m, v, c)), bits(prev))
    mask, val = oracle.changed_mask(theta, m, v, c)
    assert np.array_equal(mask.astype(bool), bt != bp)
    assert np.array_equal(val, bt)
    assert 0 < mask.sum() < mask.size


@pytest.mark.parametrize("lr,wd", [(0.1, 1.0), (0.5, 1.0), (1e-3, 0.2), (-0.1, 1.0)])
def test_changed_set_against_unfused_arrays_where_bf16_is_subnormal(lr, wd):
    """The lowest BF16 cells (|theta| < 2^-126: fp32 and BF16 subnormals) with steps of up to a
    cell and a half and a division by a decay away from 1: every intermediate here is subnormal
    or next to it, so a flushed operand or result anywhere would show."""
    hp = Hyper(step=20, lr=lr, wd=wd)
    rng = np.random.default_rng(7)
    n = 200003
    pat = (rng.integers(0, 0x40, size=n, dtype=np.uint32) << 16) | rng.integers(0, 1 << 16, size=n, dtype=np.uint32)
    theta = (pat | (rng.integers(0, 2, size=n, dtype=np.uint32) << 31)).view(np.float32).copy()
    v = (2.0 ** rng.uniform(20, 60, size=n)).astype(np.float32)
    c = oracle.derive_constants(*hp.as_args())
    c64 = c.astype(np.float64)
    step = rng.uniform(-1.5, 1.5, size=n) * 2.0 ** -133
    m = (step / abs(c64[3]) * (np.sqrt(v.astype(np.float64) / c64[1]) + c64[4]) * c64[0]).astype(np.float32)
    m[::7] = 0.0
    prev, bt, bp = _unfused_numpy(theta, m, v, c)
    assert np.array_equal(bits(oracle.invert(theta, m, v, c)), bits(prev))
    mask, val = oracle.changed_mask(theta, m, v, c)
    assert np.array_equal(mask.astype(bool), bt != bp)
    assert np.array_equal(val, bt)
    assert 0.05 < mask.mean() < 0.999
    # the range is what it claims to be: subnormal operands and results
    tiny = np.float32(2.0 ** -126)
    assert (np.abs(theta) < tiny).mean() > 0.9 and (np.abs(prev) < tiny).mean() > 0.5


def test_changed_set_zero_sign_and_nan_rules():
    c = oracle.derive_constants(100, 1e-6, 0.9, 0.999, 1e-8, 0.0)
    # +0 / -0 are different stored patterns
    th = np.float32([-0.0, 0.0, -0.0])
    m = np.float32([0.0, -0.0, -0.0])
    v = np.float32([1.0, 1.0, 1.0])
    mask, val = oracle.changed_mask(th, m, v, c)
    # -0 + +0 = +0 (changed); +0 + -0 = +0 (unchanged); -0 + -0 = -0 (unchanged)
    assert list(mask) == [1, 0, 0] and list(val) == [0x8000, 0x0000, 0x8000]
    # NaN on both sides compares equal (both 0x7FC0); NaN on one side differs
    c0 = oracle.derive_constants(100, 1e-6, 0.9, 0.999, 0.0, 0.0)
    th = np.array([np.nan, 1.0, f32_from_bits(0xFFC00001)], np.float32)
    m = np.float32([0.0, 0.0, 1.0])
    v = np.float32([1.0, 0.0, 1.0])   # second: 0/0 -> NaN reconstruction from a finite theta
    mask, val = oracle.changed_mask(th, m, v, c0)
    assert list(mask) == [0, 1, 0] and list(val) == [0x7FC0, 0x3F80, 0x7FC0]
