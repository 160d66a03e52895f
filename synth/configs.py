"""The synthetic workloads: a plan, hyper-parameters and per-tensor distributions.

These stand in for the optimizer states of Qwen3-8B / Qwen3-30B-A3B after an
RL step (public model dimensions, change density below 2 %); no trained weight
or dataset item is involved.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np
import torch

from . import plans as P
from .tensors import (Hyper, Spec, WEIGHT, NORM, calibrate_sigma_g, make_state, plant_edges,
                      routing_counts)


@dataclass
class State:
    theta: List[torch.Tensor]
    m: List[torch.Tensor]
    v: List[torch.Tensor]
    prev_bf16: List[Optional[torch.Tensor]]

    def free_prev(self):
        self.prev_bf16 = [None] * len(self.prev_bf16)


@dataclass
class Workload:
    name: str
    plan: P.Plan
    hp: Hyper
    specs: List[Spec]
    seed: int = 1234
    variant: str = "mirror"
    plant: bool = False
    plant_nonfinite: bool = False
    notes: Dict[str, object] = field(default_factory=dict)
    # alias_of[p] = tensor whose allocation p shares (distributed-optimizer slices of one shard)
    alias_of: Optional[List[int]] = None

    def materialize(self, device, tensors: Optional[List[int]] = None) -> State:
        """Generate theta_t/m_t/v_t (+BF16 theta_{t-1}) for all (or the listed) tensors."""
        n = self.plan.n_tensors
        st = State([None] * n, [None] * n, [None] * n, [None] * n)
        for p in (range(n) if tensors is None else tensors):
            d = make_state(self.plan.tensor_names[p], self.plan.numel(p), self.specs[p], self.hp,
                           self.seed, device, self.variant)
            if self.plant:
                plant_edges(d["theta"], d["m"], d["v"], self.seed + p, self.plant_nonfinite)
            st.theta[p], st.m[p], st.v[p], st.prev_bf16[p] = d["theta"], d["m"], d["v"], d["prev_bf16"]
        return st


def _is_norm(name: str) -> bool:
    return "norm" in name


def _specs(plan: P.Plan, weight: Spec = WEIGHT, norm: Spec = NORM) -> List[Spec]:
    return [norm if _is_norm(n) else weight for n in plan.tensor_names]


HP_T100 = Hyper(step=100, lr=1e-6, wd=0.01)
HP_T500 = Hyper(step=500, lr=1e-6, wd=0.01)


def config1(rows=4096, cols=4096, tp=2, seed=1234) -> Workload:
    """One q_proj-shaped matrix, column-parallel TP=2, literal generator parameters."""
    plan = P.single_matrix_plan(rows, cols, tp)
    return Workload("qwen3-8b.q_proj.tp2", plan, HP_T100, _specs(plan), seed)


def config2(tp=4, seed=1234, dims=P.QWEN3_8B, hp=HP_T100, weight: Spec = WEIGHT) -> Workload:
    """One Qwen3-8B decoder layer, TP=4 with fused qkv / gate_up and row-parallel o / down."""
    plan = P.qwen3_dense_plan(1, tp, False, dims)
    return Workload(f"qwen3-8b.layer.tp{tp}", plan, hp, _specs(plan, weight), seed)


def config3(device, n_layers=36, tp=2, seed=1234, dims=P.QWEN3_8B, with_embeddings=True,
            target=0.015) -> Workload:
    """Full Qwen3-8B-shaped state; sigma_g calibrated so the true change rate is ~1.5 %."""
    plan = P.qwen3_dense_plan(n_layers, tp, with_embeddings, dims)
    w = calibrate_sigma_g(WEIGHT, HP_T500, seed, device, target)
    wl = Workload(f"qwen3-8b.full{n_layers}.tp{tp}", plan, HP_T500, _specs(plan, w), seed)
    wl.notes["sigma_g"] = w.sigma_g
    return wl


def config3_mcore(device, tp_send=2, tp_recv=2, dp=1, n_layers=36, seed=1234, dims=P.QWEN3_8B,
                  target=0.015) -> Workload:
    """Config 3's state held the way Megatron-Core holds it: fused GQA-interleaved linear_qkv and
    fused linear_fc1 per sender TP rank, column shards of linear_proj / linear_fc2, and `dp`
    distributed-optimizer slices per shard (all slices of a shard share one allocation here)."""
    plan = P.mcore_dense_plan(n_layers, tp_send, tp_recv, True, dims, dp=dp)
    w = calibrate_sigma_g(WEIGHT, HP_T500, seed, device, target)
    wl = Workload(f"qwen3-8b.mcore.tp{tp_send}to{tp_recv}.dp{dp}.full{n_layers}", plan, HP_T500,
                  _specs(plan, w), seed)
    wl.notes.update(sigma_g=w.sigma_g, operations=len(plan.ops))
    if dp > 1:
        wl.alias_of = [(t // dp) * dp for t in range(plan.n_tensors)]
    return wl


def config4(device, n_layers=12, seed=1234, dims=P.QWEN3_30B_A3B, target=0.015,
            tokens=64, tp=4, ep=4) -> Workload:
    """Qwen3-30B-A3B-shaped slice; experts' state scaled by a Zipf routing histogram.
    tp > ep: tensor-parallel experts; tp > 4 (the KV head count): replicated KV heads."""
    plan = P.qwen3_moe_plan(n_layers, tp, ep, dims)
    w = calibrate_sigma_g(WEIGHT, HP_T500, seed, device, target)
    specs = _specs(plan, w)
    cold = 0
    E = dims["experts"]
    for l in range(n_layers):
        c = routing_counts(seed, l, E, tokens)
        mean = c.mean()
        cold += int((c == 0).sum())
        for p, name in enumerate(plan.tensor_names):
            if name.startswith(f"layers.{l}.experts."):
                e = int(name.split(".")[3])
                specs[p] = replace(w, scale=float(c[e] / mean))
    wl = Workload(f"qwen3-30b-a3b.first{n_layers}.tp{tp}ep{ep}", plan, HP_T500, specs, seed)
    wl.notes.update(sigma_g=w.sigma_g, cold_experts=cold, routing_tokens=tokens)
    return wl


def config5_points():
    """(lr, step, wd, sigma_g) sweep of the density / edge configuration."""
    pts = []
    for lr in (1e-8, 1e-7, 1e-6, 1e-5, 1e-4):
        for step in (1, 100):
            for wd in (0.01, 0.1):
                pts.append((lr, step, wd, 1e-3))
    pts.append((1e-4, 100, 0.01, 1e-2))
    return pts


def config5(lr, step, wd, sigma_g, tp=4, seed=1234, dims=P.QWEN3_8B, nonfinite=False) -> Workload:
    plan = P.qwen3_dense_plan(1, tp, False, dims)
    hp = Hyper(step=step, lr=lr, wd=wd)
    wl = Workload(f"qwen3-8b.layer.tp{tp}.lr{lr:g}.t{step}.wd{wd:g}", plan, hp,
                  _specs(plan, replace(WEIGHT, sigma_g=sigma_g)), seed, plant=True,
                  plant_nonfinite=nonfinite)
    return wl


# Reduced dimensions with the same structure (ragged widths on purpose) for
# element-by-element parity tests the oracle finishes in seconds.
SMALL_DENSE = dict(hidden=384, q_heads=8, kv_heads=4, head_dim=32, inter=1152, vocab=3000,
                   layers=2)
SMALL_MOE = dict(hidden=256, q_heads=8, kv_heads=4, head_dim=32, experts=16, moe_inter=96,
                 layers=2)
