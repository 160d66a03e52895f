"""The two-round same-cluster transfer (Section 4.3) on CPU ranks (gloo): senders hold
Megatron-Core-native TP shards, receivers hold inference TP shards; the lists come from the
oracle, travel through both rounds and are applied with the oracle; every receiver must end with
exactly the shards a single-process extract + apply of the whole plan produces."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _lists_of(plan, st, hp, oracle):
    ops = plan.ops_array()
    need = set(int(x) for x in ops[:, 0])
    zero = np.zeros(0, np.float32)
    shapes = [s if p in need else (0, 1) for p, s in enumerate(plan.tensor_shapes)]
    host = lambda lst: [lst[p].numpy() if p in need else zero for p in range(plan.n_tensors)]
    c = oracle.derive_constants(*hp.as_args())
    return oracle.extract(shapes, plan.shard_numels, ops, host(st.theta), host(st.m), host(st.v), c,
                          with_op_counts=True)


def scenario_bad_rank(scenario):
    return scenario[6] if len(scenario) > 6 else None


def _worker(rank, world, port, out, scenario):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2608_00455_b200.transfer import TwoRoundTransfer
        from synth import configs, plans
        from synth.tensors import Hyper

        tp_send, tp_recv, rank_of_sender, rank_of_receiver, lr, zero_calls = scenario[:6]
        plan = plans.mcore_dense_plan(1, tp_send, tp_recv, True, configs.SMALL_DENSE)
        owners = plans.tensor_senders(plan, tp_send)
        hp = Hyper(step=200, lr=lr, wd=0.05)
        wl = configs.Workload("xfer", plan, hp, configs._specs(plan), 321)
        st = wl.materialize("cpu")
        ops = plan.ops_array()
        xfer = TwoRoundTransfer(plan.shard_receivers, ops[:, 1], [owners[int(t)] for t in ops[:, 0]],
                                rank_of_sender, rank_of_receiver, zero_count_calls=zero_calls)
        sender = rank_of_sender.index(rank) if rank in rank_of_sender else None
        receiver = rank_of_receiver.index(rank) if rank in rank_of_receiver else None
        args = {}
        if sender is not None:
            sub = plans.sender_subplan(plan, owners, sender)
            lp, off, val, counts = _lists_of(sub, st, hp, oracle)
            args = dict(list_ptr=lp, offsets=torch.from_numpy(off.view(np.int32).copy()),
                        values=torch.from_numpy(val.view(np.int16).copy()),
                        op_counts=torch.from_numpy(counts.astype(np.int64)))
        if scenario_bad_rank(scenario) == rank:     # this sender announces one entry too many
            args["op_counts"] = args["op_counts"].clone()
            args["op_counts"][0] += 1
        if scenario_bad_rank(scenario) is not None:
            try:
                xfer.exchange(rank, sender, receiver, **args)
                out.put({"rank": rank, "raised": None})
            except RuntimeError as e:
                out.put({"rank": rank, "raised": str(e)})
            dist.barrier()
            return
        got = xfer.exchange(rank, sender, receiver, **args)
        report = {"rank": rank, "senders": sorted(got), "entries": {s: int(g.offsets.numel()) for s, g in got.items()}}
        if receiver is not None:
            # apply what arrived, sender by sender, and compare with the single-process result
            shards = [np.zeros(n, np.uint16) for n in plan.shard_numels]
            for s in sorted(got):
                g = got[s]
                oracle.apply(plan.shard_numels, g.list_ptr, g.offsets.numpy().view(np.uint32),
                             g.values.numpy().view(np.uint16), shards)
            lp, off, val, counts = _lists_of(plan, st, hp, oracle)
            want = [np.zeros(n, np.uint16) for n in plan.shard_numels]
            oracle.apply(plan.shard_numels, lp, off, val, want)
            mine = [k for k, r in enumerate(plan.shard_receivers) if r == receiver]
            report["shards_equal"] = all(np.array_equal(shards[k], want[k]) for k in mine)
            report["others_untouched"] = all(not shards[k].any() for k in range(plan.n_shards) if k not in mine)
            report["changed"] = int(sum(int(lp[k + 1] - lp[k]) for k in mine))
            # round 1 delivered c_o of every operation of every route, zeros included
            ok = True
            for s in sorted(got):
                rt = xfer.routes[s, receiver]
                ok &= np.array_equal(got[s].op_counts, counts[rt.ops].astype(np.int64))
                ok &= got[s].op_counts.size == rt.ops.size
            report["counts_equal"] = bool(ok)
            report["zero_count_ops"] = int(sum(int((g.op_counts == 0).sum()) for g in got.values()))
        out.put(report)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def _run(world, scenario, port_base):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = port_base + os.getpid() % 1500
    ps = [ctx.Process(target=_worker, args=(r, world, port, q, scenario)) for r in range(world)]
    for p in ps:
        p.start()
    reports = [q.get(timeout=300) for _ in ps]
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    return {r["rank"]: r for r in reports}


def test_two_ranks_each_sender_and_receiver():
    res = _run(2, (2, 2, [0, 1], [0, 1], 2e-6, False), 31000)
    for rank in (0, 1):
        r = res[rank]
        assert r["shards_equal"] and r["others_untouched"] and r["counts_equal"], r
        assert r["changed"] > 100 and sum(r["entries"].values()) == r["changed"]
        assert rank in r["senders"]            # the local route needs no communication


def test_disjoint_roles_two_senders_one_receiver():
    # ranks 0 and 1 hold the training shards, rank 2 the whole inference copy
    res = _run(3, (2, 1, [0, 1], [2], 2e-6, False), 33000)
    assert res[0]["senders"] == [] and res[1]["senders"] == []
    r = res[2]
    assert r["senders"] == [0, 1] and r["shards_equal"] and r["counts_equal"] and r["changed"] > 100


@pytest.mark.parametrize("zero_calls", [False, True])
def test_nothing_changed_keeps_the_schedule_aligned(zero_calls):
    # a learning rate too small to move any BF16 value: every c_o is zero, round 1 still runs for
    # every route and round 2 is either skipped on both sides or issued with empty buffers
    res = _run(2, (2, 2, [0, 1], [0, 1], 1e-12, zero_calls), 35000 + 700 * zero_calls)
    for rank in (0, 1):
        r = res[rank]
        assert r["changed"] == 0 and r["shards_equal"] and r["counts_equal"]
        assert r["zero_count_ops"] > 0 and sum(r["entries"].values()) == 0


def test_inconsistent_counts_on_one_sender_block_no_rank():
    # rank 1's counts do not add up to its lists: it stays in the schedule, announces the failure in
    # round 1 and raises after round 2; its peers raise too (nothing usable arrived from it), and
    # every process reaches the final barrier - a rank that left early would hang the others
    res = _run(3, (2, 2, [0, 1], [1, 2], 2e-6, False, 1), 37000)
    assert "counts announce" in res[1]["raised"]
    assert "sender 1 reported inconsistent lists" in res[2]["raised"]
    assert res[0]["raised"] is None          # a sender with consistent lists is not affected


def test_schedule_is_static_and_symmetric():
    from paper_2608_00455_b200.transfer import TwoRoundTransfer
    from synth import configs, plans
    plan = plans.mcore_dense_plan(2, 4, 2, True, dict(configs.SMALL_DENSE, vocab=3008))
    owners = plans.tensor_senders(plan, 4)
    ops = plan.ops_array()
    x = TwoRoundTransfer(plan.shard_receivers, ops[:, 1], [owners[int(t)] for t in ops[:, 0]], range(4), [4, 5])
    covered = np.zeros(len(plan.ops), np.int32)
    for (s, r), rt in x.routes.items():
        covered[rt.ops] += 1
        assert np.all(np.diff(rt.ops) > 0)                              # plan order
        assert all(owners[plan.ops[o][0]] == s and plan.shard_receivers[plan.ops[o][1]] == r for o in rt.ops)
        assert rt.contiguous and np.array_equal(x.sender_ops[s][rt.local_ops], rt.ops)
    assert np.all(covered == 1)                                          # every operation travels exactly once


def test_counts_that_disagree_with_the_lists_stop_the_sender():
    # announced counts and payload length must match before anything is sent
    from paper_2608_00455_b200.transfer import TwoRoundTransfer
    x = TwoRoundTransfer([0, 0], [0, 1], [0, 0], [0], [0])            # one sender, one receiver, same rank
    lp = np.array([0, 3, 5], np.uint64)
    off = torch.arange(5, dtype=torch.int32)
    val = torch.arange(5, dtype=torch.int16)
    got = x.exchange(0, 0, 0, lp, off, val, torch.tensor([3, 2]))
    assert got[0].list_ptr.tolist() == [0, 3, 5] and torch.equal(got[0].offsets, off)
    # the local route reports both sides of the failure
    with pytest.raises(RuntimeError, match="counts announce 4 entries, lists hold 5; sender 0 reported"):
        x.exchange(0, 0, 0, lp, off, val, torch.tensor([3, 1]))
