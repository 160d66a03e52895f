"""Adversarial inputs for the extract kernel's conservative screen: theta within a few fp32
ulps of a BF16 rounding boundary and update terms of about the same size, so that the
decision "cannot have changed" is taken right at its threshold.  Bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from synth import plans
from synth.tensors import Hyper

pytestmark = pytest.mark.gpu


def _near_boundary_state(n, hp: Hyper, seed, spread_ulps=24, with_specials=True):
    """theta = BF16 tie point +- a few ulps; m, v chosen so |lr*u| is 0..2*spread ulps of theta."""
    rng = np.random.default_rng(seed)
    upper = rng.integers(0x3000, 0x4800, size=n, dtype=np.uint32)         # exponents 2^-31 .. 2^17
    sign = rng.integers(0, 2, size=n, dtype=np.uint32) << 31
    delta = rng.integers(-spread_ulps, spread_ulps + 1, size=n).astype(np.int64)
    bits = ((upper.astype(np.int64) << 16) + 0x8000 + delta).astype(np.uint32) | sign
    theta = bits.view(np.float32).copy()
    ulp = np.spacing(np.abs(theta)).astype(np.float64)
    want_step = rng.uniform(0, 2 * spread_ulps, size=n) * ulp * rng.choice([-1.0, 1.0], size=n)
    c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
    v = np.abs(rng.standard_normal(n) * 1e-6).astype(np.float32) + np.float32(1e-12)
    # lr * (m/bc1) / (sqrt(v/bc2) + eps) ~= want_step  =>  m
    m = (want_step / c[3] * (np.sqrt(v.astype(np.float64) / c[1]) + c[4]) * c[0]).astype(np.float32)
    if with_specials:
        k = n // 64
        v[:k] = 0.0                                   # eps-dominated denominators
        m[k:2 * k] = 0.0
        v[2 * k:3 * k] = np.float32(1e-42)            # subnormal second moment
        theta[3 * k:3 * k + 16] = 0.0
        m[3 * k + 16:3 * k + 32] = np.float32(np.inf)
        v[3 * k + 32:3 * k + 48] = -1.0
        theta[3 * k + 48:3 * k + 64] = np.float32(np.nan)
    return theta, m, v


@pytest.mark.parametrize("hp", [
    Hyper(step=500, lr=1e-6, wd=0.01),        # bc1 == 1, decay == 1
    Hyper(step=100, lr=1e-6, wd=0.01),        # bc1 != 1, decay == 1
    Hyper(step=500, lr=1e-4, wd=0.1),         # bc1 == 1, decay != 1
    Hyper(step=1, lr=3e-4, wd=0.3),           # both divisions, extreme bias correction
    Hyper(step=7, lr=1e-3, wd=0.0, eps=0.0),  # eps == 0
    Hyper(step=50, lr=1e-5, wd=5.0, beta1=0.5, beta2=0.9),
], ids=lambda h: f"t{h.step}-lr{h.lr:g}-wd{h.wd:g}-eps{h.eps:g}")
def test_screen_threshold_cases_match_oracle(hp):
    rows, cols = 4096, 2048
    n = rows * cols
    theta, m, v = _near_boundary_state(n, hp, seed=hp.step)
    plan = plans.single_matrix_plan(rows, cols, 2)
    c = oracle.derive_constants(*hp.as_args())
    want = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), [theta], [m], [v], c)
    lay = dte.Layout.from_plan(plan, 0)
    d = lay.new_delta(n)
    t, mm, vv = (torch.from_numpy(a).cuda() for a in (theta, m, v))
    dte.dte_extract_delta(lay, lay.source_tables([t], [mm], [vv]), *hp.as_args(), d)
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    lp, off, val = d.to_host()
    assert np.array_equal(lp, want[0])
    assert np.array_equal(off, want[1])
    assert np.array_equal(val, want[2])
    frac = int(lp[-1]) / n
    assert 0.05 < frac < 0.95, frac            # the cases really straddle the decision


@pytest.mark.parametrize("hp", [
    Hyper(step=500, lr=1e-6, wd=0.01),                 # no division by bc1 or decay
    Hyper(step=3, lr=1e-3, wd=0.2),                    # both
    Hyper(step=100, lr=1e-6, wd=0.01),                 # bc1 only
    Hyper(step=500, lr=1e-4, wd=0.1),                  # decay only
    Hyper(step=7, lr=1e-3, wd=0.0, eps=0.0),           # eps == 0
    Hyper(step=20, lr=0.5, wd=1.5),                    # decay = 0.25
    Hyper(step=20, lr=-1e-3, wd=0.5),                  # negative learning rate, decay > 1
    Hyper(step=2, lr=1e-2, wd=0.01, beta1=0.0, beta2=0.5, eps=1e-30),
], ids=lambda h: f"t{h.step}-lr{h.lr:g}-wd{h.wd:g}-eps{h.eps:g}")
def test_random_bit_patterns_match_oracle(hp):
    """theta, m, v drawn as raw 32-bit patterns: every exponent, subnormals, Inf, NaN, negative
    second moments.  Nothing here is a plausible optimizer state; the point is that the screen
    never clears an element whose exact evaluation would differ."""
    rows, cols = 2048, 4096
    n = rows * cols
    rng = np.random.default_rng(99 + hp.step)
    theta = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32).view(np.float32)
    m = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32).view(np.float32)
    vb = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    vb[: n // 2] &= 0x7FFFFFFF                        # half of the second moments non-negative
    v = vb.view(np.float32)
    # a band of moderate magnitudes so that part of the data takes the screened path at all
    k = n // 4
    theta[:k] = (rng.standard_normal(k) * 0.02).astype(np.float32)
    m[:k] = (rng.standard_normal(k) * 10.0 ** rng.uniform(-12, 2, k)).astype(np.float32)
    v[:k] = np.abs(rng.standard_normal(k) * 10.0 ** rng.uniform(-20, 2, k)).astype(np.float32)
    plan = plans.single_matrix_plan(rows, cols, 2)
    c = oracle.derive_constants(*hp.as_args())
    with np.errstate(all="ignore"):
        want = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), [theta], [m], [v], c)
    lay = dte.Layout.from_plan(plan, 0)
    d = lay.new_delta(n)
    t, mm, vv = (torch.from_numpy(a.copy()).cuda() for a in (theta, m, v))
    dte.dte_extract_delta(lay, lay.source_tables([t], [mm], [vv]), *hp.as_args(), d)
    torch.cuda.synchronize()
    lp, off, val = d.to_host()
    assert np.array_equal(lp, want[0]) and np.array_equal(off, want[1]) and np.array_equal(val, want[2])
    assert 0.3 < int(lp[-1]) / n <= 1.0


def _wide_exponent_threshold_state(n, hp: Hyper, seed):
    """Like the near-boundary state, but over EVERY binade of theta and of the second moment:
    theta a few ulps off a BF16 tie point with any exponent (subnormals included), v with any
    exponent, m solved (in double) so that the update is 1/8 .. 8 times the distance to the tie -
    where that needs an m, m-hat or u beyond fp32's range it overflows or underflows, on purpose."""
    rng = np.random.default_rng(seed)
    upper = rng.integers(0x0000, 0x7F80, size=n, dtype=np.uint32)
    sign = rng.integers(0, 2, size=n, dtype=np.uint32) << 31
    delta = rng.integers(-40, 41, size=n).astype(np.int64)
    bits = np.clip((upper.astype(np.int64) << 16) + 0x8000 + delta, 0, 0x7F7FFFFF).astype(np.uint32) | sign
    theta = bits.view(np.float32).copy()
    vexp = rng.integers(1, 255, size=n, dtype=np.uint32)
    v = ((vexp << 23) | rng.integers(0, 1 << 23, size=n, dtype=np.uint32)).view(np.float32).copy()
    with np.errstate(all="ignore"):
        dist = np.abs(delta).astype(np.float64) * np.spacing(np.abs(theta)).astype(np.float64)
        dist = np.where(dist == 0, np.spacing(np.abs(theta)).astype(np.float64), dist)
        factor = 2.0 ** rng.uniform(-3, 3, size=n)
        c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
        lr = c[3] if c[3] != 0 else 1.0
        m64 = dist * factor / abs(lr) * (np.sqrt(v.astype(np.float64) / c[1]) + c[4]) * c[0]
        m = (m64 * rng.choice([-1.0, 1.0], size=n)).astype(np.float32)
    return theta, m, v


@pytest.mark.parametrize("hp", [
    Hyper(step=500, lr=1e-6, wd=0.01),
    Hyper(step=3, lr=1e-3, wd=0.2),
    Hyper(step=100, lr=1e-6, wd=0.01),
    Hyper(step=500, lr=1e-4, wd=0.1),
    Hyper(step=7, lr=1e-3, wd=0.0, eps=0.0),
    Hyper(step=20, lr=-1e-3, wd=0.5),
    Hyper(step=2, lr=1e-2, wd=0.01, beta1=0.0, beta2=0.5, eps=1e-30),
    Hyper(step=40, lr=1e-12, wd=0.0, eps=1e-20),       # tiny lr: huge m-hat and u for a visible step
    Hyper(step=40, lr=30.0, wd=0.0, eps=1e-3),         # large lr: tiny m-hat and u
], ids=lambda h: f"t{h.step}-lr{h.lr:g}-wd{h.wd:g}-eps{h.eps:g}")
def test_threshold_cases_in_every_binade_match_oracle(hp):
    rows, cols = 2048, 4096
    n = rows * cols
    theta, m, v = _wide_exponent_threshold_state(n, hp, seed=1000 + hp.step)
    plan = plans.single_matrix_plan(rows, cols, 2)
    c = oracle.derive_constants(*hp.as_args())
    with np.errstate(all="ignore"):
        want = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), [theta], [m], [v], c)
    lay = dte.Layout.from_plan(plan, 0)
    d = lay.new_delta(n)
    t, mm, vv = (torch.from_numpy(a.copy()).cuda() for a in (theta, m, v))
    dte.dte_extract_delta(lay, lay.source_tables([t], [mm], [vv]), *hp.as_args(), d)
    torch.cuda.synchronize()
    lp, off, val = d.to_host()
    assert np.array_equal(lp, want[0]) and np.array_equal(off, want[1]) and np.array_equal(val, want[2])
    assert 0.02 < int(lp[-1]) / n < 0.98
