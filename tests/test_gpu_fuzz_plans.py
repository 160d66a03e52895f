"""Parity fuzz over seeded random transfer plans: arbitrary hyper-rectangles (odd shapes, row /
column / grid splits, one-row pieces, stacked destinations with gaps, replication, unread
regions), random hyper-parameters per case.  Lists, counters, per-operation counts and applied
shards must equal the oracle's bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from gpu_util import assert_lists_equal, oracle_extract, run_extract
from synth import configs, plans
from synth.tensors import Hyper, Spec

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(40))
def test_random_plan_matches_the_oracle(seed):
    plan = plans.random_plan(1000 + seed)
    rng = np.random.default_rng(seed)
    hp = Hyper(step=int(rng.integers(1, 600)), lr=float(10.0 ** rng.uniform(-6.5, -3.5)),
               wd=float(rng.choice([0.0, 0.01, 0.1])))
    wl = configs.Workload(f"fuzz{seed}", plan, hp, [Spec()] * plan.n_tensors, 7000 + seed, plant=bool(seed % 2))
    st = wl.materialize("cuda")
    lay, d = run_extract(plan, st, hp)
    assert d.status_bits() == 0
    got = d.to_host()
    want = oracle_extract(plan, st, hp)
    assert_lists_equal(got, want, plan)
    cnt = d.counters.cpu().numpy()
    assert cnt[0] == int(want[0][-1]) and cnt[1] == plan.total_scanned_elements()
    # per-operation counts (round 1 of the transfer), plan order, zeros included
    ops = plan.ops_array()
    need = set(int(x) for x in ops[:, 0])
    zero = np.zeros(0, np.float32)
    shapes = [s if p in need else (0, 1) for p, s in enumerate(plan.tensor_shapes)]
    host = lambda lst: [lst[p].cpu().numpy() if p in need else zero for p in range(plan.n_tensors)]
    want_counts = oracle.extract(shapes, plan.shard_numels, ops, host(st.theta), host(st.m), host(st.v),
                                 oracle.derive_constants(*hp.as_args()), with_op_counts=True)[3]
    assert np.array_equal(dte.dte_op_counts(lay, d).cpu().numpy().astype(np.uint64), want_counts)
    # apply onto canaries: listed slots take the values, every other slot keeps its canary
    shards = [torch.full((n,), 0x5A5A, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply(lay, d, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    ref = [np.full(n, 0x5A5A, np.uint16) for n in plan.shard_numels]
    oracle.apply(plan.shard_numels, *want, ref)
    for k in range(plan.n_shards):
        assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), ref[k]), plan.shard_names[k]
