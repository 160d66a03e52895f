"""Pins for the Megatron-Core-native source layouts (fused GQA-interleaved linear_qkv, fused
linear_fc1, sender-side TP shards, distributed-optimizer slices): the plan, evaluated densely
and through the oracle, must reproduce the textbook conversion - unpack the fused tensors into
q/k/v/o/gate/up/down (the paper's Eq. 14-17), then shard for the receivers with chunk / cat."""
import numpy as np
import pytest
import torch

import oracle
from synth import configs, plans

D = configs.SMALL_DENSE
SENTINEL = 0x7ABC


def _canonical(seed):
    g = torch.Generator().manual_seed(seed)
    h, hd, hq, hkv, F, V = D["hidden"], D["head_dim"], D["q_heads"], D["kv_heads"], D["inter"], D["vocab"]
    shapes = dict(q=(hq * hd, h), k=(hkv * hd, h), v=(hkv * hd, h), o=(h, hq * hd), gate=(F, h), up=(F, h),
                  down=(h, F), q_norm=(hd,), k_norm=(hd,), ln1=(h,), ln2=(h,), emb=(V, h), head=(V, h))
    return {k: torch.randint(-30000, 30000, s, generator=g, dtype=torch.int16) for k, s in shapes.items()}


def _mcore_sources(c, P):
    """Sender-side tensors of one layer (+ embeddings) from the canonical ones, in plan order."""
    hd, hq, hkv, F, V = D["head_dim"], D["q_heads"], D["kv_heads"], D["inter"], D["vocab"]
    g = hq // hkv
    out = []
    for s in range(P):
        groups = range(s * hkv // P, (s + 1) * hkv // P)
        qkv = torch.cat([torch.cat([c["q"][j * g * hd:(j + 1) * g * hd], c["k"][j * hd:(j + 1) * hd],
                                    c["v"][j * hd:(j + 1) * hd]]) for j in groups])
        out.append(qkv)
        out.append(c["o"].chunk(P, 1)[s].contiguous())
        out.append(torch.cat([c["gate"].chunk(P, 0)[s], c["up"].chunk(P, 0)[s]]))
        out.append(c["down"].chunk(P, 1)[s].contiguous())
    out += [c["q_norm"], c["k_norm"], c["ln1"], c["ln2"]]
    for s in range(P):
        out.append(c["emb"].chunk(P, 0)[s].contiguous())
        out.append(c["head"].chunk(P, 0)[s].contiguous())
    return out


def _textbook_receivers(c, R):
    out = []
    for r in range(R):
        out.append(torch.cat([c["q"].chunk(R, 0)[r], c["k"].chunk(R, 0)[r], c["v"].chunk(R, 0)[r]]))
        out.append(c["o"].chunk(R, 1)[r])
        out.append(torch.cat([c["gate"].chunk(R, 0)[r], c["up"].chunk(R, 0)[r]]))
        out.append(c["down"].chunk(R, 1)[r])
        out += [c["q_norm"], c["k_norm"], c["ln1"], c["ln2"]]
        out += [c["emb"].chunk(R, 0)[r], c["head"].chunk(R, 0)[r]]
    return [t.reshape(-1) for t in out]


@pytest.mark.parametrize("P,R,dp", [(1, 2, 1), (2, 2, 1), (2, 4, 1), (4, 2, 1), (1, 1, 1), (2, 2, 3), (2, 4, 2), (4, 2, 2)])
def test_mcore_plan_reproduces_the_textbook_conversion(P, R, dp):
    plan = plans.mcore_dense_plan(1, P, R, True, D, dp=dp)
    c = _canonical(P * 10 + R)
    src = _mcore_sources(c, P)
    assert len(src) * dp == plan.n_tensors
    if dp > 1:      # each owner holds only its flat slice: everything else is a sentinel
        sliced = []
        for t, full in enumerate(src):
            for d in range(dp):
                lo, hi = plan.slice_ranges[t * dp + d]
                buf = torch.full((full.numel(),), SENTINEL, dtype=torch.int16)
                buf[lo:hi] = full.reshape(-1)[lo:hi]
                sliced.append(buf.reshape(full.shape))
            assert plan.slice_ranges[t * dp][0] == 0 and plan.slice_ranges[t * dp + dp - 1][1] == full.numel()
        src = sliced
    shards = [torch.full((n,), -1, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, src, shards)
    want = _textbook_receivers(c, R)
    assert len(want) == plan.n_shards
    for k, w in enumerate(want):
        assert torch.equal(shards[k], w), plan.shard_names[k]


@pytest.mark.parametrize("P,R,dp", [(2, 4, 1), (4, 2, 1), (2, 2, 3)])
def test_mcore_plan_covers_every_receiver_slot_exactly_once(P, R, dp):
    plan = plans.mcore_dense_plan(1, P, R, True, D, dp=dp)
    rng = np.random.default_rng(1)
    th = [(rng.standard_normal(plan.numel(p)) * 0.02).astype(np.float32) for p in range(plan.n_tensors)]
    mm = [np.full(plan.numel(p), 0.5, np.float32) for p in range(plan.n_tensors)]
    c = oracle.derive_constants(1, 8.0, 0.5, 0.5, 0.0, 0.0)       # every element changes
    if dp > 1:      # elements outside an owner's slice must never be read: make them unchanged
        for p in range(plan.n_tensors):
            lo, hi = plan.slice_ranges[p]
            keep = np.zeros(plan.numel(p), bool)
            keep[lo:hi] = True
            mm[p][~keep] = 0.0
    vv = [m.copy() for m in mm]
    # m = v = 0 with eps = 0 gives NaN (changed); use eps > 0 for the masked elements instead
    c = oracle.derive_constants(1, 8.0, 0.5, 0.5, 1e-3, 0.0)
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    for k, n in enumerate(plan.shard_numels):
        assert np.array_equal(off[int(lp[k]):int(lp[k + 1])], np.arange(n, dtype=np.uint32)), plan.shard_names[k]


def test_restrict_to_flat_range_partitions_an_operation():
    op = (0, 0, 2, 3, 6, 10, 100, 10, 1, 0)          # rows 2..7, cols 3..12 of a 16-column source
    n1 = 16
    seen = {}
    cuts = [0, 37, 40, 41, 77, 96, 200]
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        for piece in plans.restrict_to_flat_range(op, n1, lo, hi):
            _, _, a0, a1, e0, e1, base, ld, r0, r1 = piece
            assert (r1 == 0 and e1 == ld) or e0 == 1
            for u0 in range(a0, a0 + e0):
                for u1 in range(a1, a1 + e1):
                    assert lo <= u0 * n1 + u1 < hi
                    j = base + (u0 - a0 + r0) * ld + (u1 - a1 + r1)
                    assert (u0, u1) not in seen
                    seen[(u0, u1)] = j
    want = {(u0, u1): 100 + (u0 - 2 + 1) * 10 + (u1 - 3) for u0 in range(2, 8) for u1 in range(3, 13)}
    assert seen == want
