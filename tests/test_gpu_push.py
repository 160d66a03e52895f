"""Same-cluster transfer fused into the extract's tail (Section 4.3): the kernel that orders the
changed entries also stores every receiver's share straight into that receiver's landing buffers,
and a closing kernel delivers list boundaries, per-operation counts (plan order, zeros included)
and - last - the status block.  One GPU stands in for the cluster: the "peers" are separate
allocations on the same device, reached with the same plain stores a peer mapping would get.
Everything a receiver ends up with is compared with the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from synth import configs, plans
from synth.tensors import Hyper
from gpu_util import assert_lists_equal, initial_shards, oracle_extract

pytestmark = pytest.mark.gpu


def _oracle_with_counts(plan, st, hp):
    c = oracle.derive_constants(*hp.as_args())
    host = lambda lst: [x.cpu().numpy() for x in lst]
    return oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), host(st.theta), host(st.m),
                          host(st.v), c, with_op_counts=True)


def _push(plan, st, hp, capacities=None, epoch=7, skip=()):
    lay = dte.Layout.from_plan(plan, 0)
    R = lay.num_receivers
    d = lay.new_delta(lay.num_elements)
    targets = []
    for r in range(R):
        cap = lay.num_elements if capacities is None else capacities[r]
        targets.append(None if r in skip else dte.PushTarget(lay.num_lists, cap, lay.receiver_num_ops(r), "cuda"))
        if targets[-1] is not None:
            targets[-1].offsets.fill_(-1)
            targets[-1].op_counts.fill_(-1)
    dte.dte_extract_delta_push(lay, lay.source_tables(st.theta, st.m, st.v), *hp.as_args(), d, targets, epoch)
    torch.cuda.synchronize()
    return lay, d, targets


def _check_receiver(plan, lay, t, r, want, epoch, st=None):
    """Receiver r's buffers against the oracle's lists of r's shards and counts of r's operations."""
    lp_w, off_w, val_w, cnt_w = want
    mine = [k for k, rr in enumerate(plan.shard_receivers) if rr == r]
    status = t.status.cpu().numpy().astype(np.uint64)
    n = int(sum(int(lp_w[k + 1] - lp_w[k]) for k in mine))
    assert status.tolist() == [n, epoch, 0, lay.receiver_num_ops(r)]
    lp = t.list_ptr.cpu().numpy().astype(np.uint64)
    assert lp[0] == 0 and lp[-1] == n
    off = t.offsets[:n].cpu().numpy().view(np.uint32)
    val = t.values[:n].cpu().numpy().view(np.uint16)
    for k in range(plan.n_shards):
        a, b = int(lp[k]), int(lp[k + 1])
        if k in mine:
            c, e = int(lp_w[k]), int(lp_w[k + 1])
            assert b - a == e - c, plan.shard_names[k]
            assert np.array_equal(off[a:b], off_w[c:e]) and np.array_equal(val[a:b], val_w[c:e]), plan.shard_names[k]
        else:
            assert a == b                      # lists of other receivers come out empty
    ops_r = [o for o, op in enumerate(plan.ops) if plan.shard_receivers[op[1]] == r]
    assert np.array_equal(t.op_counts[:len(ops_r)].cpu().numpy().astype(np.uint64), cnt_w[ops_r])
    return mine, n


@pytest.mark.parametrize("name", ["dense_tp4", "moe_tp4_ep4", "dense_tp2_small_layout"])
def test_push_delivers_every_receivers_lists_counts_and_status(name):
    plan = {"dense_tp4": lambda: plans.qwen3_dense_plan(3, 4, True, configs.SMALL_DENSE),
            "moe_tp4_ep4": lambda: plans.qwen3_moe_plan(2, 4, 4, configs.SMALL_MOE),
            "dense_tp2_small_layout": lambda: plans.qwen3_dense_plan(1, 2, False, configs.SMALL_DENSE)}[name]()
    hp = Hyper(step=100, lr=1e-5, wd=0.01)
    wl = configs.Workload(name, plan, hp, configs._specs(plan), 31)
    st = wl.materialize("cuda")
    for p in range(0, plan.n_tensors, 5):          # some tensors do not change: zero counts, empty lists
        st.m[p].zero_()
        st.v[p].zero_()
    want = _oracle_with_counts(plan, st, hp)
    lay, d, targets = _push(plan, st, hp)
    assert d.status_bits() == 0
    assert_lists_equal(d.to_host(), want[:3], plan)          # the sender keeps complete lists
    assert (want[3] == 0).sum() > 0
    shards = initial_shards(plan, st)
    host = [s.cpu().numpy().view(np.uint16).copy() for s in shards]
    oracle.apply(plan.shard_numels, *want[:3], host)
    for r, t in enumerate(targets):
        mine, n = _check_receiver(plan, lay, t, r, want, 7)
        # the receiver waits for the epoch and applies its share to the tensors it holds
        dte.dte_push_wait(t, 7, timeout_ms=1000)
        tab = lay.shard_table([s if k in mine else None for k, s in enumerate(shards)])
        dte.dte_apply(lay, t.delta(), tab)
        torch.cuda.synchronize()
        assert t.counters.cpu().tolist() == [n, 0, 0, 0]
    for k in range(plan.n_shards):
        assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), host[k]), plan.shard_names[k]


def test_push_full_dimension_layer_large_layout_path():
    # config 2 at full dimensions: 20 9xx tiles, so the three-launch gather and its scan of the
    # receivers' slice starts are used (the small plans above take the one-launch gather)
    wl = configs.config2()
    st = wl.materialize("cuda")
    want = _oracle_with_counts(wl.plan, st, wl.hp)
    lay, d, targets = _push(wl.plan, st, wl.hp, capacities=[1 << 20] * 4, epoch=3)
    assert lay.last_launch()["tiles"] > 4096 and d.status_bits() == 0
    assert_lists_equal(d.to_host(), want[:3], wl.plan)
    for r, t in enumerate(targets):
        _check_receiver(wl.plan, lay, t, r, want, 3)


def test_push_when_nothing_changed_still_delivers_zero_counts_and_the_status_block():
    plan = plans.qwen3_dense_plan(2, 4, True, configs.SMALL_DENSE)
    hp = Hyper(step=100, lr=1e-3, wd=0.0)
    wl = configs.Workload("still", plan, hp, configs._specs(plan), 5)
    st = wl.materialize("cuda")
    st.m = [torch.zeros_like(x) for x in st.m]
    st.v = [torch.zeros_like(x) for x in st.v]
    lay, d, targets = _push(plan, st, hp, epoch=41)
    assert d.total() == 0 and d.status_bits() == 0
    for r, t in enumerate(targets):
        assert t.status.cpu().tolist() == [0, 41, 0, lay.receiver_num_ops(r)]
        assert int(t.list_ptr.abs().sum()) == 0 and int(t.op_counts[:t.n_ops].abs().sum()) == 0
    # and a second version on the same layout and targets: the epoch moves on
    wl2 = configs.Workload("moves", plan, Hyper(step=101, lr=1e-5, wd=0.01), configs._specs(plan), 6)
    st2 = wl2.materialize("cuda")
    want = _oracle_with_counts(plan, st2, wl2.hp)
    dte.dte_extract_delta_push(lay, lay.source_tables(st2.theta, st2.m, st2.v), *wl2.hp.as_args(), d, targets, 42)
    torch.cuda.synchronize()
    for r, t in enumerate(targets):
        _check_receiver(plan, lay, t, r, want, 42)


def test_push_target_too_small_and_skipped_receivers():
    plan = plans.qwen3_dense_plan(2, 4, True, configs.SMALL_DENSE)
    hp = Hyper(step=100, lr=1e-4, wd=0.01)
    wl = configs.Workload("tight", plan, hp, configs._specs(plan), 9)
    st = wl.materialize("cuda")
    want = _oracle_with_counts(plan, st, hp)
    per_recv = [int(sum(int(want[0][k + 1] - want[0][k]) for k, rr in enumerate(plan.shard_receivers) if rr == r))
                for r in range(4)]
    assert min(per_recv) > 200
    caps = [per_recv[0], 100, per_recv[2] + 5, per_recv[3]]        # receiver 1's buffers are too small
    lay, d, targets = _push(plan, st, hp, capacities=caps, skip=(3,))
    _check_receiver(plan, lay, targets[0], 0, want, 7)
    _check_receiver(plan, lay, targets[2], 2, want, 7)
    t = targets[1]
    assert t.status.cpu().tolist() == [per_recv[1], 7, dte.DTE_DEV_OVERFLOW, lay.receiver_num_ops(1)]
    assert int(t.list_ptr[-1]) == per_recv[1]                       # exact sizes, so it can grow
    # such a share is refused by apply
    dte.dte_push_wait(t, 7)
    shard = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply(lay, t.delta(), lay.shard_table(shard))
    torch.cuda.synchronize()
    assert all(int(s.abs().sum()) == 0 for s in shard)


def test_push_wait_gives_up_after_its_time_limit_and_the_context_stays_usable():
    t = dte.PushTarget(4, 16, 1, "cuda")
    t.counters.fill_(5)
    dte.dte_push_wait(t, epoch=99, timeout_ms=20)                  # nothing will ever write epoch 99
    torch.cuda.synchronize()
    c = t.counters.cpu().tolist()
    assert c[0] == 0 and c[2] == (dte.DTE_DEV_TIMEOUT | dte.DTE_DEV_OVERFLOW)
    x = torch.arange(10, device="cuda").sum().item()               # the device still answers
    assert x == 45


def test_push_needs_consecutive_shards_per_receiver():
    p = plans.Plan()
    a = p.add_tensor("a", (64, 64))
    k0 = p.add_shard("r0.a", 0, 1024)
    k1 = p.add_shard("r1.a", 1, 2048)
    k2 = p.add_shard("r0.b", 0, 1024)
    p.add_op(a, k0, (0, 0), (16, 64), 0, 64, (0, 0))
    p.add_op(a, k1, (16, 0), (32, 64), 0, 64, (0, 0))
    p.add_op(a, k2, (48, 0), (16, 64), 0, 64, (0, 0))
    lay = dte.Layout.from_plan(p, 0)
    z = torch.zeros(64 * 64, dtype=torch.float32, device="cuda")
    targets = [dte.PushTarget(3, 64, lay.receiver_num_ops(r), "cuda") for r in range(2)]
    with pytest.raises(dte.DteError) as e:
        dte.dte_extract_delta_push(lay, lay.source_tables([z], [z], [z]), 1, 1e-3, 0.9, 0.999, 1e-8, 0.0,
                                   lay.new_delta(64), targets, 1)
    assert e.value.status == 2


def test_receiver_ids_beyond_the_push_tables_leave_the_layout_usable_without_push():
    """`receiver` is informational for extract and apply; ids above 65534 (2^32 - 1 included, which
    must not wrap to a receiver count of zero) only switch the push off."""
    for rid in (65535, 0xFFFFFFFF):
        p = plans.Plan()
        a = p.add_tensor("a", (64, 64))
        k0 = p.add_shard("r0.a", 0, 2048)
        k1 = p.add_shard("far.a", rid, 2048)
        p.add_op(a, k0, (0, 0), (32, 64), 0, 64, (0, 0))
        p.add_op(a, k1, (32, 0), (32, 64), 0, 64, (0, 0))
        lay = dte.Layout.from_plan(p, 0)
        assert lay.num_receivers == 0
        theta = torch.randn(64 * 64, device="cuda") * 0.02
        m = torch.randn(64 * 64, device="cuda") * 1e-2
        v = torch.rand(64 * 64, device="cuda") * 1e-6
        d = lay.new_delta(64 * 64)
        dte.dte_extract_delta(lay, lay.source_tables([theta], [m], [v]), 10, 1e-3, 0.9, 0.999, 1e-8, 0.0, d)
        torch.cuda.synchronize()
        assert d.status_bits() == 0 and d.total() > 0
        with pytest.raises(dte.DteError) as e:
            dte.dte_extract_delta_push(lay, lay.source_tables([theta], [m], [v]), 10, 1e-3, 0.9, 0.999, 1e-8, 0.0,
                                       d, [], 1)
        assert e.value.status == 2


def test_push_into_a_second_gpus_memory_when_there_is_one():
    """The intended deployment: the landing buffers live on the receiver's GPU and the sender's
    gather kernel stores into them through peer access.  Needs two GPUs that can reach each other
    (this test is skipped on a single-GPU machine; everything else about the push is covered above
    with landing buffers on the sender's own GPU)."""
    if torch.cuda.device_count() < 2 or not torch.cuda.can_device_access_peer(0, 1):
        pytest.skip("needs two GPUs with peer access")
    torch.zeros(8, device="cuda:0").to("cuda:1")               # lets torch enable peer access 0 -> 1
    plan = plans.qwen3_dense_plan(2, 2, True, configs.SMALL_DENSE)
    hp = Hyper(step=100, lr=1e-5, wd=0.01)
    wl = configs.Workload("p2p", plan, hp, configs._specs(plan), 77)
    st = wl.materialize("cuda:0")
    want = _oracle_with_counts(plan, st, hp)
    send = dte.Layout.from_plan(plan, 0)
    recv = dte.Layout.from_plan(plan, 1)                       # the receiver compiles the same plan
    d = send.new_delta(send.num_elements)
    # receiver 0 stays on the sender's GPU, receiver 1 is the second GPU
    targets = [dte.PushTarget(send.num_lists, send.num_elements, send.receiver_num_ops(0), "cuda:0"),
               dte.PushTarget(send.num_lists, send.num_elements, send.receiver_num_ops(1), "cuda:1")]
    mine = [k for k, r in enumerate(plan.shard_receivers) if r == 1]
    with torch.cuda.device(1):
        shards = [torch.zeros(n, dtype=torch.int16, device="cuda:1") if k in mine else None
                  for k, n in enumerate(plan.shard_numels)]
        s1 = torch.cuda.current_stream(1)
        torch.cuda.synchronize(1)
        # the receiver waits (at most 5 s) on its own GPU while the sender works on the other
        dte.dte_push_wait(targets[1], 9, timeout_ms=5000, stream=s1)
        dte.dte_apply(recv, targets[1].delta(), recv.shard_table(shards), stream=s1)
    dte.dte_extract_delta_push(send, send.source_tables(st.theta, st.m, st.v), *hp.as_args(), d, targets, 9)
    torch.cuda.synchronize(0)
    torch.cuda.synchronize(1)
    _check_receiver(plan, send, targets[0], 0, want, 9)
    _check_receiver(plan, send, targets[1], 1, want, 9)
    assert targets[1].counters.cpu().tolist()[2] == 0
    lp_w, off_w, val_w, _ = want
    for k in mine:
        exp = np.zeros(plan.shard_numels[k], np.uint16)
        seg = slice(int(lp_w[k]), int(lp_w[k + 1]))
        exp[off_w[seg]] = val_w[seg]
        assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), exp), plan.shard_names[k]
