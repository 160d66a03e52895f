"""Seeded synthetic optimizer state (inputs only; none of the method's arithmetic).

Each tensor gets theta_{t-1}, a gradient and prior moments from a seeded
generator, then one *forward* AdamW step (Eq. 1 and Eq. 9) in fp32 with every
operation rounded separately.  What comes out is what a trainer would hold
after step t: theta_t, m_t, v_t, plus BF16(theta_{t-1}) for initialising
receiver buffers.  The same code runs on CPU (oracle pins) and on the GPU
(parity tests, benchmark); CPU and GPU random streams differ, so parity tests
copy the device tensors to the host instead of regenerating them.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, replace
from typing import Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Hyper:
    step: int = 100
    lr: float = 1e-6
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    wd: float = 0.01

    def as_args(self):
        return (self.step, self.lr, self.beta1, self.beta2, self.eps, self.wd)


@dataclass(frozen=True)
class Spec:
    """Distribution of one tensor's state before the step (sigma = std dev)."""
    mu: float = 0.0
    sigma_theta: float = 0.02
    sigma_g: float = 1e-3
    sigma_m: float = 1e-4
    sigma_v: float = 1e-6
    scale: float = 1.0      # multiplies g, m_{t-1} and sqrt(v_{t-1}); 0 => exactly zero state


WEIGHT = Spec()
NORM = Spec(mu=1.0)


def tensor_seed(seed: int, name: str) -> int:
    h = hashlib.sha256(f"{seed}:{name}".encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 62) - 1)


def _f(x: float) -> float:
    return float(np.float32(x))


def forward_adamw(theta_prev, g, m_prev, v_prev, hp: Hyper, variant: str = "mirror"):
    """One AdamW step in fp32, each operation its own rounding (Eq. 1, Eq. 9).

    variant "mirror": theta_t = fl(fl(theta_{t-1}*(1-lr*wd)) - fl(lr*u));
    variant "trainer": theta_t = theta_{t-1} - lr*(u + wd*theta_{t-1}).
    Scalars derived in double and rounded once to fp32.
    """
    b1, b2 = _f(hp.beta1), _f(hp.beta2)
    omb1, omb2 = _f(1.0 - hp.beta1), _f(1.0 - hp.beta2)
    bc1 = _f(1.0 - hp.beta1 ** hp.step)
    bc2 = _f(1.0 - hp.beta2 ** hp.step)
    lr, eps, wd = _f(hp.lr), _f(hp.eps), _f(hp.wd)
    decay = _f(1.0 - hp.lr * hp.wd)
    m = m_prev * b1
    m += g * omb1
    v = v_prev * b2
    v += (g * g) * omb2
    u = (m / bc1) / (torch.sqrt(v / bc2) + eps)
    if variant == "mirror":
        theta = theta_prev * decay - u * lr
    elif variant == "trainer":
        theta = theta_prev - (u + theta_prev * wd) * lr
    else:
        raise ValueError(variant)
    return theta, m, v


CHUNK = 1 << 25


def make_state(name: str, numel: int, spec: Spec, hp: Hyper, seed: int, device,
               variant: str = "mirror", keep_prev_fp32: bool = False):
    """Returns dict(theta, m, v: fp32[numel]; prev_bf16: bf16[numel] [, prev: fp32])."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(tensor_seed(seed, name))
    out = dict(theta=torch.empty(numel, dtype=torch.float32, device=dev),
               m=torch.empty(numel, dtype=torch.float32, device=dev),
               v=torch.empty(numel, dtype=torch.float32, device=dev),
               prev_bf16=torch.empty(numel, dtype=torch.bfloat16, device=dev))
    if keep_prev_fp32:
        out["prev"] = torch.empty(numel, dtype=torch.float32, device=dev)
    for lo in range(0, numel, CHUNK):
        n = min(CHUNK, numel - lo)
        sl = slice(lo, lo + n)

        def rn():
            return torch.randn(n, dtype=torch.float32, device=dev, generator=gen)

        prev = rn() * _f(spec.sigma_theta) + _f(spec.mu)
        if spec.scale == 0.0:
            # the draws are still consumed so that streams do not depend on `scale`
            rn(); rn(); rn()
            g = torch.zeros_like(prev)
            m0 = torch.zeros_like(prev)
            v0 = torch.zeros_like(prev)
        else:
            s = _f(spec.scale)
            g = rn() * _f(spec.sigma_g * s)
            m0 = rn() * _f(spec.sigma_m * s)
            v0 = (rn() * _f(spec.sigma_v * s * s)).abs_()
        theta, m, v = forward_adamw(prev, g, m0, v0, hp, variant)
        out["theta"][sl] = theta
        out["m"][sl] = m
        out["v"][sl] = v
        out["prev_bf16"][sl] = prev.to(torch.bfloat16)
        if keep_prev_fp32:
            out["prev"][sl] = prev
    return out


def true_change_rate(spec: Spec, hp: Hyper, seed: int, device, n: int = 1 << 20,
                     variant: str = "mirror") -> float:
    """Fraction of a sample whose BF16 pattern differs between theta_{t-1} and theta_t."""
    st = make_state("calibration", n, spec, hp, seed, device, variant)
    cur = st["theta"].to(torch.bfloat16).view(torch.int16)
    return float((cur != st["prev_bf16"].view(torch.int16)).float().mean().item())


def calibrate_sigma_g(spec: Spec, hp: Hyper, seed: int, device, target: float = 0.015,
                      lo: float = 1e-5, hi: float = 1.0, iters: int = 18,
                      variant: str = "mirror") -> Spec:
    """Bisection (log scale) on sigma_g so that the sample's true change rate ~ target.

    The rate grows with sigma_g until |u| saturates; if even `hi` stays below
    the target, `hi` is returned.
    """
    if true_change_rate(replace(spec, sigma_g=hi), hp, seed, device, variant=variant) < target:
        return replace(spec, sigma_g=hi)
    a, b = np.log(lo), np.log(hi)
    for _ in range(iters):
        mid = 0.5 * (a + b)
        r = true_change_rate(replace(spec, sigma_g=float(np.exp(mid))), hp, seed, device,
                             variant=variant)
        if r < target:
            a = mid
        else:
            b = mid
    return replace(spec, sigma_g=float(np.exp(0.5 * (a + b))))


def routing_counts(seed: int, layer: int, n_experts: int = 128, tokens: int = 64, top_k: int = 8,
                   zipf_s: float = 1.1) -> np.ndarray:
    """Tokens routed to each expert: top_k distinct experts per token, Zipf-skewed."""
    rng = np.random.default_rng(tensor_seed(seed, f"routing.{layer}") % (1 << 32))
    perm = rng.permutation(n_experts)
    w = 1.0 / np.arange(1, n_experts + 1) ** zipf_s
    w /= w.sum()
    counts = np.zeros(n_experts, np.int64)
    for _ in range(tokens):
        pick = rng.choice(n_experts, size=top_k, replace=False, p=w)
        counts[perm[pick]] += 1
    return counts


# ---- planted edge values -------------------------------------------------------

def _bits(vals):
    return torch.tensor(np.asarray(vals, dtype=np.uint32).view(np.int32), dtype=torch.int32)


def plant_edges(theta: torch.Tensor, m: torch.Tensor, v: torch.Tensor, seed: int,
                with_nonfinite: bool = False) -> int:
    """Overwrite a fixed index pattern with rounding ties, zeros, extremes and subnormals.

    Patterns (fp32 bit patterns of theta): BF16 ties with even and odd upper
    half and one fp32 ulp either side; +-0; values near +-65504; the BF16
    overflow threshold 0x7F7F8000 +- 1; fp32 subnormals; combined with v = 0
    (m != 0 and m == 0).  Returns how many positions were planted.
    """
    n = theta.numel()
    pats = [0x3F808000, 0x3F807FFF, 0x3F808001, 0x3F818000, 0x3F817FFF, 0x3F818001,
            0xBF808000, 0xBF818000, 0x00000000, 0x80000000,
            0x477FE000, 0xC77FE000, 0x477FDFFF, 0x477FE001,
            0x7F7F8000, 0x7F7F7FFF, 0x7F7F8001, 0xFF7F8000, 0x7F7FFFFF,
            0x00000001, 0x00008000, 0x00007FFF, 0x80000001, 0x007FFFFF, 0x00800000,
            0x3C008000, 0x3C018000, 0x3C00FFFF]
    if with_nonfinite:
        pats += [0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00001, 0x7F800001]
    rng = np.random.default_rng(tensor_seed(seed, "plant") % (1 << 32))
    reps = 4
    k = len(pats) * reps
    if n < 4 * k:
        return 0
    idx = torch.from_numpy(np.sort(rng.choice(n, size=k, replace=False))).to(theta.device)
    tb = _bits(np.tile(np.asarray(pats, dtype=np.uint32), reps)).to(theta.device)
    theta.view(torch.int32)[idx] = tb
    # moment variants cycle with the repetition number
    rep = torch.arange(k, device=theta.device) // len(pats)
    mi, vi = m[idx].clone(), v[idx].clone()
    vi[rep == 1] = 0.0                       # v = 0, m as drawn
    vi[rep == 2] = 0.0
    mi[rep == 2] = 0.0                       # v = 0 and m = 0
    mi[rep == 3] = -mi[rep == 3].abs()       # force the other sign of the update
    m[idx] = mi
    v[idx] = vi
    return k
