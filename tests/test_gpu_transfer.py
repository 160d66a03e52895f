"""The transfer schedule driven by the real kernels on one GPU: extract on a sender's plan,
per-operation counts from the device, both rounds (a rank that plays sender and receiver moves
its route locally), apply of what arrived - against a direct extract + apply of the whole plan
and against the oracle's counts."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from gpu_util import oracle_extract, run_extract
from paper_2608_00455_b200.transfer import TwoRoundTransfer
from synth import configs, plans
from synth.tensors import Hyper

pytestmark = pytest.mark.gpu


def test_senders_to_one_receiver_through_both_rounds():
    tp_send = 2
    plan = plans.mcore_dense_plan(1, tp_send, 1, True, configs.SMALL_DENSE)
    owners = plans.tensor_senders(plan, tp_send)
    hp = Hyper(step=200, lr=2e-6, wd=0.05)
    wl = configs.Workload("xfer", plan, hp, configs._specs(plan), 321)
    st = wl.materialize("cuda")
    ops = plan.ops_array()
    op_sender = [owners[int(t)] for t in ops[:, 0]]

    # reference: the whole plan in one extract + apply
    lay_all, d_all = run_extract(plan, st, hp)
    want = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply(lay_all, d_all, lay_all.shard_table(want))
    want_lists = oracle_extract(plan, st, hp)
    full_counts = oracle.extract(plan.tensor_shapes, plan.shard_numels, ops, [t.cpu().numpy() for t in st.theta],
                                 [t.cpu().numpy() for t in st.m], [t.cpu().numpy() for t in st.v],
                                 oracle.derive_constants(*hp.as_args()), with_op_counts=True)[3]
    assert np.array_equal(d_all.to_host()[1], want_lists[1])

    shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    total = 0
    for s in range(tp_send):
        # this process plays sender s and the receiver in turn: a one-sender schedule over s's plan
        sub = plans.sender_subplan(plan, owners, s)
        sub_ops = sub.ops_array()
        xfer = TwoRoundTransfer(plan.shard_receivers, sub_ops[:, 1], [0] * len(sub_ops), [0], [0])
        theta = [t if owners[p] == s else None for p, t in enumerate(st.theta)]
        lay = dte.Layout.from_plan(sub, 0)
        d = lay.new_delta(lay.num_elements)
        dte.dte_extract_delta(lay, lay.source_tables(theta, [m if owners[p] == s else None for p, m in enumerate(st.m)],
                                                     [v if owners[p] == s else None for p, v in enumerate(st.v)]),
                              *hp.as_args(), d)
        counts = dte.dte_op_counts(lay, d)
        torch.cuda.synchronize()
        mine = np.nonzero(np.asarray(op_sender) == s)[0]
        assert np.array_equal(counts.cpu().numpy(), full_counts[mine].astype(np.int64))
        got = xfer.exchange(0, 0, 0, d.list_ptr.cpu().numpy().astype(np.uint64), d.offsets, d.values, counts, "cuda")
        g = got[0]
        assert np.array_equal(g.op_counts, full_counts[mine].astype(np.int64))
        total += int(g.offsets.numel())
        dte.dte_apply(lay_all, dte.Delta.wrap(g.list_ptr, g.offsets, g.values), lay_all.shard_table(shards))
    torch.cuda.synchronize()
    assert total == d_all.total()
    for k in range(plan.n_shards):
        assert torch.equal(shards[k], want[k]), plan.shard_names[k]
