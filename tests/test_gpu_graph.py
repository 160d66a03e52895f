"""Extract + apply captured once into a CUDA graph and replayed on new state: after a first
ordinary call (which sizes the staging buffer and uploads the pointer tables) the calls only
enqueue memsets and kernels, so a stream capture records them; replays must track the data."""
import numpy as np
import pytest
import torch

import paper_2608_00455_b200 as dte
from gpu_util import assert_lists_equal, oracle_extract
from synth import configs, plans
from synth.tensors import Hyper

pytestmark = pytest.mark.gpu


def test_captured_step_replays_on_new_state():
    plan = plans.qwen3_dense_plan(1, 2, True, configs.SMALL_DENSE)
    hp = Hyper(step=100, lr=1e-5, wd=0.01)
    a = configs.Workload("g0", plan, hp, configs._specs(plan), 41).materialize("cuda")
    b = configs.Workload("g1", plan, hp, configs._specs(plan), 42).materialize("cuda")
    lay = dte.Layout.from_plan(plan, 0)
    d = lay.new_delta(lay.num_elements)
    # static buffers the graph reads; their contents change between replays
    th = [t.clone() for t in a.theta]; mm = [t.clone() for t in a.m]; vv = [t.clone() for t in a.v]
    tabs = lay.source_tables(th, mm, vv)
    shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    tab = lay.shard_table(shards)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        dte.dte_extract_delta(lay, tabs, *hp.as_args(), d)       # ordinary first call
        dte.dte_apply(lay, d, tab)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            dte.dte_extract_delta(lay, tabs, *hp.as_args(), d)
            dte.dte_apply(lay, d, tab)
    for st in (b, a, b):
        for dst, src in zip(th + mm + vv, st.theta + st.m + st.v):
            dst.copy_(src)
        for s in shards:
            s.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert d.status_bits() == 0
        want = oracle_extract(plan, st, hp)
        assert_lists_equal(d.to_host(), want, plan)
        lp, off, val = want
        for k in range(plan.n_shards):
            exp = np.zeros(plan.shard_numels[k], np.uint16)
            seg = slice(int(lp[k]), int(lp[k + 1]))
            exp[off[seg]] = val[seg]
            assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), exp)
