"""GPU parity on Megatron-Core-native source layouts: GQA-interleaved fused linear_qkv, fused
linear_fc1, sender-side TP shards (more or fewer than the receivers) and distributed-optimizer
slices, bit-exact against the oracle (lists and applied shards)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from synth import configs, plans
from synth.tensors import Hyper
from gpu_util import assert_lists_equal, oracle_extract, run_extract

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("P,R,dp", [(2, 4, 1), (4, 2, 1), (2, 2, 3), (1, 2, 5)])
def test_mcore_native_sources(P, R, dp):
    plan = plans.mcore_dense_plan(2, P, R, True, configs.SMALL_DENSE, dp=dp)
    wl = configs.Workload(f"mcore.tp{P}to{R}.dp{dp}", plan, Hyper(step=100, lr=1e-5, wd=0.01),
                          configs._specs(plan), 31)
    st = wl.materialize("cuda")
    if dp > 1:
        # an owner holds only its slice: poison everything else so that a stray read would show
        for p in range(plan.n_tensors):
            lo, hi = plan.slice_ranges[p]
            for a in (st.theta, st.m, st.v):
                a[p][:lo] = float("nan")
                a[p][hi:] = float("nan")
    lay, d = run_extract(plan, st, wl.hp)
    assert d.status_bits() == 0
    got = d.to_host()
    want = oracle_extract(plan, st, wl.hp)
    assert_lists_equal(got, want, plan)
    assert 0 < int(got[0][-1]) < lay.num_elements // 5
    assert not np.any(got[2] == 0x7FC0)                 # no poisoned element was emitted
    bufs = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply(lay, d, lay.shard_table(bufs))
    torch.cuda.synchronize()
    host = [np.zeros(n, np.uint16) for n in plan.shard_numels]
    oracle.apply(plan.shard_numels, *want, host)
    for k in range(plan.n_shards):
        assert np.array_equal(bufs[k].cpu().numpy().view(np.uint16), host[k]), plan.shard_names[k]
