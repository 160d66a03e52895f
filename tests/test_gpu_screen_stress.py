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


def _run_and_compare(plan, hp, theta, m, v, n):
    """Lists bit-exact against the oracle, and the count of broken reconstructions too (every
    element whose reconstruction is NaN or overflowed has to reach the exact path to be counted)."""
    c = oracle.derive_constants(*hp.as_args())
    with np.errstate(all="ignore"):
        *want, odd = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), [theta], [m], [v], c,
                                    with_nonfinite=True)
    lay = dte.Layout.from_plan(plan, 0)
    d = lay.new_delta(n)
    t, mm, vv = (torch.from_numpy(a.copy()).cuda() for a in (theta, m, v))
    dte.dte_extract_delta(lay, lay.source_tables([t], [mm], [vv]), *hp.as_args(), d)
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    lp, off, val = d.to_host()
    assert np.array_equal(lp, want[0])
    assert np.array_equal(off, want[1])
    assert np.array_equal(val, want[2])
    assert int(d.counters[3].item()) == int(odd)
    return int(lp[-1]) / n, int(odd)


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
    frac, _ = _run_and_compare(plan, hp, theta, m, v, n)
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
    frac, odd = _run_and_compare(plan, hp, theta, m, v, n)
    assert odd > n // 8                               # NaN operands, negative second moments, overflows
    assert 0.3 < frac <= 1.0


def _wide_exponent_threshold_state(n, hp: Hyper, seed, upper_range=(0x0000, 0x7F80)):
    """Like the near-boundary state, but over EVERY binade of theta and of the second moment:
    theta a few ulps off a BF16 tie point with any exponent (subnormals included), v with any
    exponent, m solved (in double) so that the update is 1/8 .. 8 times the distance to the tie -
    where that needs an m, m-hat or u beyond fp32's range it overflows or underflows, on purpose."""
    rng = np.random.default_rng(seed)
    upper = rng.integers(upper_range[0], upper_range[1], size=n, dtype=np.uint32)
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
    frac, _ = _run_and_compare(plan, hp, theta, m, v, n)
    assert 0.02 < frac < 0.98


@pytest.mark.parametrize("hp", [
    Hyper(step=500, lr=1e-6, wd=0.01),                 # theta beyond the last BF16 tie point casts to Inf, and so does its reconstruction
    Hyper(step=20, lr=30.0, wd=0.0, eps=1e-3),         # theta + lr * u overflows
    Hyper(step=20, lr=0.5, wd=1.0),                    # the division by decay = 0.5 overflows
    Hyper(step=20, lr=30.0, wd=0.01),                  # both can
    Hyper(step=20, lr=-4.0, wd=1.0),                   # decay = 5: a finite sum shrinks, one that overflowed stays infinite
], ids=lambda h: f"t{h.step}-lr{h.lr:g}-wd{h.wd:g}-eps{h.eps:g}")
def test_reconstructions_at_the_top_of_the_range_match_oracle(hp):
    """theta in the last binades of fp32 (up to the largest finite value, past the last BF16 tie
    point), steps from negligible to several times theta: reconstructions that stay finite, that
    overflow in the sum, and that overflow in the division by decay.  The lists and the count of
    overflowed reconstructions must both match."""
    rows, cols = 2048, 2048
    n = rows * cols
    rng = np.random.default_rng(4242 + hp.step + int(hp.lr * 10) % 97)
    upper = rng.integers(0x7E00, 0x7F80, size=n, dtype=np.uint32)
    low = rng.integers(0, 1 << 16, size=n, dtype=np.uint32)
    sign = rng.integers(0, 2, size=n, dtype=np.uint32) << 31
    theta = ((upper << 16) | low | sign).view(np.float32).copy()
    theta[: n // 16] = np.float32(3.4028234663852886e38) * rng.choice([-1.0, 1.0], size=n // 16).astype(np.float32)
    v = (2.0 ** rng.uniform(-20, 20, size=n)).astype(np.float32)
    c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
    with np.errstate(all="ignore"):
        step = np.abs(theta).astype(np.float64) * 2.0 ** rng.uniform(-30, 4, size=n) * rng.choice([-1.0, 1.0], size=n)
        m = (step / abs(c[3]) * (np.sqrt(v.astype(np.float64) / c[1]) + c[4]) * c[0]).astype(np.float32)
    plan = plans.single_matrix_plan(rows, cols, 2)
    frac, odd = _run_and_compare(plan, hp, theta, m, v, n)
    if hp.lr >= 0.5 or hp.lr < 0:
        assert odd > n // 100, odd            # overflows really happen
    assert 0.001 < frac <= 1.0


@pytest.mark.parametrize("hp", [
    Hyper(step=20, lr=0.1, wd=1.0),                    # decay = 0.9
    Hyper(step=20, lr=0.25, wd=1.0),                   # 0.75
    Hyper(step=20, lr=0.5, wd=1.0),                    # 0.5: the division moves theta by as much as theta
    Hyper(step=20, lr=0.999, wd=1.0),                  # 0.001
    Hyper(step=20, lr=-0.1, wd=1.0),                   # 1.1
    Hyper(step=20, lr=-4.0, wd=1.0),                   # 5
    Hyper(step=20, lr=1e-3, wd=0.2),                   # 0.9998
    Hyper(step=20, lr=1e-5, wd=1.0),                   # 0.99999
], ids=lambda h: f"lr{h.lr:g}-wd{h.wd:g}")
@pytest.mark.parametrize("still", [False, True], ids=["step", "no-step"])
def test_division_by_decay_where_bf16_is_subnormal_matches_oracle(hp, still):
    """theta in the fp32-subnormal, BF16-subnormal and first normal binades, where a BF16 rounding
    cell is as wide as the values in it and the rounding error of the division is absolute, not
    relative: a division by a decay well away from 1 leaves many of these elements in their cell,
    so the decision is taken at its threshold there (in the normal range such a decay changes
    everything).  Once with steps of about the distance to the tie point, once with m = 0, which
    leaves the division alone."""
    rows, cols = 2048, 2048
    n = rows * cols
    seed = 77 + int(abs(hp.lr) * 1e5) % 1000
    theta, m, v = _wide_exponent_threshold_state(n, hp, seed=seed, upper_range=(0x0000, 0x0100))
    # half of the elements anywhere in the sixteen lowest BF16 cells instead of next to a tie point:
    # there the distance to the tie is of the size of the division's shift
    rng = np.random.default_rng(seed + 1)
    k = n // 2
    bits = (rng.integers(0x0000, 0x0010, size=k, dtype=np.uint32) << 16) | rng.integers(0, 1 << 16, size=k, dtype=np.uint32)
    theta[:k] = (bits | (rng.integers(0, 2, size=k, dtype=np.uint32) << 31)).view(np.float32)
    # ... with steps of up to a cell and a half, so that theta and theta + step can sit at opposite
    # ends of one cell (a step of next to nothing relative to anything normal, but here the sum
    # is up to three times theta, and the division's shift grows with it)
    c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
    v[:k] = (2.0 ** rng.uniform(20, 60, size=k)).astype(np.float32)
    step = rng.uniform(-1.5, 1.5, size=k) * 2.0 ** -133
    m[:k] = (step / abs(c[3]) * (np.sqrt(v[:k].astype(np.float64) / c[1]) + c[4]) * c[0]).astype(np.float32)
    if still:
        m[:] = 0.0
    plan = plans.single_matrix_plan(rows, cols, 2)
    frac, _ = _run_and_compare(plan, hp, theta, m, v, n)
    assert 0.01 < frac < 1.0


@pytest.mark.parametrize("hp", [
    Hyper(step=500, lr=1e-6, wd=0.01),
    Hyper(step=3, lr=1e-3, wd=0.2),
    Hyper(step=20, lr=1e-3, wd=1.0),                   # decay = 0.999: a shift of a quarter of a BF16 cell
    Hyper(step=20, lr=-1e-3, wd=0.5),
    Hyper(step=7, lr=1e-3, wd=0.0, eps=0.0),
], ids=lambda h: f"t{h.step}-lr{h.lr:g}-wd{h.wd:g}-eps{h.eps:g}")
def test_steps_of_every_relative_size_in_every_binade_match_oracle(hp):
    """theta anywhere (every binade, every position in its BF16 cell), the step from 2^-30 of
    theta to 16 times theta and of either sign: elements that cannot change, that sit at the
    threshold, that cancel to zero or flip their sign."""
    rows, cols = 2048, 4096
    n = rows * cols
    rng = np.random.default_rng(31337 + hp.step)
    upper = rng.integers(0x0000, 0x7F80, size=n, dtype=np.uint32)
    theta = ((upper << 16) | rng.integers(0, 1 << 16, size=n, dtype=np.uint32)
             | (rng.integers(0, 2, size=n, dtype=np.uint32) << 31)).view(np.float32).copy()
    v = (2.0 ** rng.uniform(-60, 60, size=n)).astype(np.float32)
    c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
    with np.errstate(all="ignore"):
        step = np.abs(theta).astype(np.float64) * 2.0 ** rng.uniform(-30, 4, size=n) * rng.choice([-1.0, 1.0], size=n)
        step[: n // 32] = -theta[: n // 32].astype(np.float64)            # exact cancellation
        m = (step / c[3] * (np.sqrt(v.astype(np.float64) / c[1]) + c[4]) * c[0]).astype(np.float32)
    plan = plans.single_matrix_plan(rows, cols, 2)
    frac, _ = _run_and_compare(plan, hp, theta, m, v, n)
    assert 0.2 < frac < 0.9


def _random_hyper(rng) -> Hyper:
    """Hyper-parameters from all over the accepted range (lr * wd < 1, betas in [0, 1), eps >= 0)."""
    lr = float(10.0 ** rng.uniform(-10, 1)) * (1.0 if rng.random() < 0.85 else -1.0)
    wd = float(rng.choice([0.0, 10.0 ** rng.uniform(-4, 0.3)]))
    if lr * wd >= 0.999:
        wd = 0.5 / abs(lr)
    eps = float(rng.choice([0.0, 1e-8, 10.0 ** rng.uniform(-30, -1)]))
    beta1 = float(rng.choice([0.0, 0.9, rng.uniform(0.0, 0.9999)]))
    beta2 = float(rng.choice([0.5, 0.999, rng.uniform(0.1, 0.99999)]))
    step = int(rng.choice([1, 2, 10, 100, 500, 5000, int(rng.integers(1, 20000))]))
    return Hyper(step=step, lr=lr, wd=wd, beta1=beta1, beta2=beta2, eps=eps)


@pytest.mark.parametrize("seed", range(32))
def test_random_hyperparameters_match_oracle(seed):
    """The screen's constants are derived from the call's hyper-parameters on the host; here those
    are random, and the state mixes the adversarial kinds above: threshold cases in every binade,
    raw bit patterns, the lowest BF16 cells with steps of about a cell, and plausible weights."""
    rng = np.random.default_rng(9000 + seed)
    hp = _random_hyper(rng)
    rows, cols = 1024, 2048
    n = rows * cols
    q = n // 4
    theta, m, v = _wide_exponent_threshold_state(n, hp, seed=seed)
    # raw bit patterns
    for a in (theta, m, v):
        a[q:2 * q] = rng.integers(0, 1 << 32, size=q, dtype=np.uint64).astype(np.uint32).view(np.float32)
    v[q:q + q // 2] = np.abs(v[q:q + q // 2])
    c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
    with np.errstate(all="ignore"):
        # the sixteen lowest BF16 cells, steps of up to a cell and a half
        bits = (rng.integers(0, 0x10, size=q, dtype=np.uint32) << 16) | rng.integers(0, 1 << 16, size=q, dtype=np.uint32)
        theta[2 * q:3 * q] = (bits | (rng.integers(0, 2, size=q, dtype=np.uint32) << 31)).view(np.float32)
        v[2 * q:3 * q] = (2.0 ** rng.uniform(20, 60, size=q)).astype(np.float32)
        step = rng.uniform(-1.5, 1.5, size=q) * 2.0 ** -133
        m[2 * q:3 * q] = (step / abs(c[3]) * (np.sqrt(v[2 * q:3 * q].astype(np.float64) / c[1]) + c[4]) * c[0]).astype(np.float32)
        # plausible weights and moments
        theta[3 * q:] = (rng.standard_normal(n - 3 * q) * 0.02).astype(np.float32)
        m[3 * q:] = (rng.standard_normal(n - 3 * q) * 1e-4).astype(np.float32)
        v[3 * q:] = np.abs(rng.standard_normal(n - 3 * q) * 1e-6).astype(np.float32)
    plan = plans.single_matrix_plan(rows, cols, 2)
    _run_and_compare(plan, hp, theta, m, v, n)


@pytest.mark.parametrize("seed", range(8))
def test_random_learning_rates_and_weight_decays_per_group_match_oracle(seed):
    """Four tensors in four parameter groups with a learning rate and a weight decay each: groups
    whose decay rounds to 1 next to groups whose decay is far from it, in one call (the kernel then
    takes every constant, the screen's included, from the tile's group)."""
    rng = np.random.default_rng(12000 + seed)
    base = _random_hyper(rng)
    lrs, wds = [], []
    for g in range(4):
        h = _random_hyper(rng)
        lrs.append(h.lr if g else 1e-6)          # group 0: lr * wd below 2^-25, decay == 1
        wds.append(h.wd if g else 0.01)
    rows, cols = 512, 2048
    n = rows * cols
    plan = plans.Plan()
    for g in range(4):
        t = plan.add_tensor(f"w{g}", (rows, cols))
        for r in range(2):
            k = plan.add_shard(f"w{g}.{r}", r, n // 2)
            plan.add_op(t, k, (r * rows // 2, 0), (rows // 2, cols), 0, cols, (0, 0))
    thetas, ms, vs = [], [], []
    for g in range(4):
        hp = Hyper(step=base.step, lr=lrs[g], wd=wds[g], beta1=base.beta1, beta2=base.beta2, eps=base.eps)
        theta, m, v = _wide_exponent_threshold_state(n, hp, seed=100 * seed + g)
        q = n // 2
        theta[q:] = (rng.standard_normal(n - q) * 0.02).astype(np.float32)
        m[q:] = (rng.standard_normal(n - q) * 1e-4).astype(np.float32)
        v[q:] = np.abs(rng.standard_normal(n - q) * 1e-6).astype(np.float32)
        thetas.append(theta); ms.append(m); vs.append(v)
    consts = np.stack([oracle.derive_constants(base.step, lrs[g], base.beta1, base.beta2, base.eps, wds[g])
                       for g in range(4)])
    with np.errstate(all="ignore"):
        *want, odd = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), thetas, ms, vs, consts,
                                    with_nonfinite=True)
    lay = dte.Layout.from_plan(plan, 0, tensor_groups=[0, 1, 2, 3])
    d = lay.new_delta(4 * n)
    dev = lambda lst: [torch.from_numpy(a.copy()).cuda() for a in lst]
    tabs = lay.source_tables(dev(thetas), dev(ms), dev(vs))
    dte.dte_extract_delta_groups(lay, tabs, base.step, base.beta1, base.beta2, base.eps, lrs, wds, d)
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    lp, off, val = d.to_host()
    assert np.array_equal(lp, want[0]) and np.array_equal(off, want[1]) and np.array_equal(val, want[2])
    assert int(d.counters[3].item()) == int(odd)


@pytest.mark.parametrize("hp", [
    Hyper(step=500, lr=1e-6, wd=0.01),
    Hyper(step=100, lr=1e-3, wd=0.0),
    Hyper(step=3, lr=1e-3, wd=0.2),
    Hyper(step=20, lr=-1e-3, wd=0.5),
], ids=lambda h: f"t{h.step}-lr{h.lr:g}-wd{h.wd:g}")
def test_large_steps_that_land_on_a_tie_point_match_oracle(hp):
    """Steps solved so that the reconstruction lands within two ulps of a BF16 tie point: from a
    theta several times smaller (of either sign), and from a theta in a cell next to that tie, where
    the decision hangs on the last bits of the sum."""
    rows, cols = 2048, 2048
    n = rows * cols
    rng = np.random.default_rng(555 + hp.step)
    upper = rng.integers(0x2000, 0x5F00, size=n, dtype=np.uint32)
    delta = rng.integers(-2, 3, size=n).astype(np.int64)
    land = (((upper.astype(np.int64) << 16) + 0x8000 + delta).astype(np.uint32)
            | (rng.integers(0, 2, size=n, dtype=np.uint32) << 31)).view(np.float32)
    theta = (land.astype(np.float64) * rng.uniform(-0.25, 0.25, size=n)).astype(np.float32)
    # half of the elements: theta already in the cell next to the tie, so that both outcomes occur
    near = rng.random(n) < 0.5
    theta[near] = (land[near].astype(np.float64) * (1.0 + rng.uniform(-3e-3, 3e-3, size=int(near.sum())))).astype(np.float32)
    v = (2.0 ** rng.uniform(-40, 40, size=n)).astype(np.float32)
    c = oracle.derive_constants(*hp.as_args()).astype(np.float64)
    with np.errstate(all="ignore"):
        step = land.astype(np.float64) * c[2] - theta.astype(np.float64)      # (theta + step) / decay = land
        m = (step / c[3] * (np.sqrt(v.astype(np.float64) / c[1]) + c[4]) * c[0]).astype(np.float32)
    plan = plans.single_matrix_plan(rows, cols, 2)
    frac, _ = _run_and_compare(plan, hp, theta, m, v, n)
    assert 0.3 < frac < 0.999
