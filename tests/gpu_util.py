"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI and the
oracle on the same (device-generated, host-copied) inputs."""
import numpy as np
import torch

import oracle
import paper_2608_00455_b200 as dte
from synth import plans as P


def run_extract(plan, st, hp, capacity=None, layout=None, delta=None):
    lay = layout or dte.Layout.from_plan(plan, 0)
    if capacity is None:
        capacity = lay.num_elements
    d = delta or lay.new_delta(capacity)
    tabs = lay.source_tables(st.theta, st.m, st.v)
    dte.dte_extract_delta(lay, tabs, *hp.as_args(), d)
    torch.cuda.synchronize()
    return lay, d


def oracle_extract(plan, st, hp, tensors=None, with_nonfinite=False):
    """Oracle on host copies.  With `tensors`, only those source tensors are evaluated
    (the other tensors' operations are dropped from the plan handed to the oracle)."""
    c = oracle.derive_constants(*hp.as_args())
    ops = plan.ops_array()
    if tensors is not None:
        keep = np.isin(ops[:, 0], np.asarray(tensors))
        ops = ops[keep]
    need = set(int(x) for x in ops[:, 0])
    zero = np.zeros(0, np.float32)
    shapes = [s if p in need else (0, 1) for p, s in enumerate(plan.tensor_shapes)]

    def host(lst):
        return [lst[p].cpu().numpy() if p in need else zero for p in range(plan.n_tensors)]

    return oracle.extract(shapes, plan.shard_numels, ops, host(st.theta), host(st.m), host(st.v), c,
                          with_nonfinite=with_nonfinite)


def assert_lists_equal(got, want, plan=None, lists=None):
    lp_g, off_g, val_g = got
    lp_w, off_w, val_w = want
    ks = range(len(lp_w) - 1) if lists is None else lists
    for k in ks:
        a, b = int(lp_g[k]), int(lp_g[k + 1])
        c, d = int(lp_w[k]), int(lp_w[k + 1])
        name = plan.shard_names[k] if plan is not None else k
        assert b - a == d - c, f"list {name}: {b - a} entries, oracle {d - c}"
        assert np.array_equal(off_g[a:b], off_w[c:d]), f"offsets of list {name}"
        assert np.array_equal(val_g[a:b], val_w[c:d]), f"values of list {name}"
    if lists is None:
        assert np.array_equal(lp_g, lp_w)


def initial_shards(plan, st, device="cuda"):
    """Receiver buffers holding remapped BF16(true theta_{t-1}) (int16 bit patterns)."""
    shards = [torch.zeros(n, dtype=torch.int16, device=device) for n in plan.shard_numels]
    P.scatter_dense(plan, [None if x is None else x.view(torch.int16) for x in st.prev_bf16], shards)
    return shards


def expected_shards(plan, st, device="cuda"):
    """Remapped BF16(theta_t) by dense slicing (library cast; no NaN in these workloads)."""
    shards = [torch.zeros(n, dtype=torch.int16, device=device) for n in plan.shard_numels]
    P.scatter_dense(plan, [x.to(torch.bfloat16).view(torch.int16) for x in st.theta], shards)
    return shards


# ---- whole-workload parity, streamed ----------------------------------------------------------

def plan_components(plan):
    """Groups of source tensors and the lists they fill, closed under "feeds the same list": the
    oracle can run on one group alone and produce those lists completely."""
    parent = list(range(plan.n_tensors + plan.n_shards))

    def find(x):
        while parent[x] != x:
            parent[x] = parent[parent[x]]
            x = parent[x]
        return x

    for o in plan.ops:
        a, b = find(int(o[0])), find(plan.n_tensors + int(o[1]))
        if a != b:
            parent[a] = b
    groups = {}
    for o in plan.ops:
        g = groups.setdefault(find(int(o[0])), (set(), set()))
        g[0].add(int(o[0]))
        g[1].add(int(o[1]))
    return [(sorted(t), sorted(k)) for t, k in groups.values()]


def full_oracle_parity(wl, st, delta, shards_before=None, shards_after=None, threads=None, budget_bytes=24e9):
    """EVERY list of the workload against the oracle, and (given the receivers' buffers before and
    after the GPU's apply) every receiver tensor against the oracle's apply from the same start.

    The state stays on the GPU; one group of tensors at a time is copied to the host (at most
    `budget_bytes` in flight) and handed to a pool of host threads that each run the plain
    single-threaded oracle on it.  Lists no operation feeds must be empty.  Returns
    (lists compared, entries compared, the oracle's entry count c_o of every operation in plan
    order)."""
    import os
    import threading
    from concurrent.futures import ThreadPoolExecutor

    plan = wl.plan
    threads = threads or (os.cpu_count() or 4)
    lp_g, off_g, val_g = delta.to_host()
    consts = oracle.derive_constants(*wl.hp.as_args())
    all_ops = plan.ops_array()
    comps = sorted(plan_components(plan), key=lambda c: -sum(plan.numel(p) for p in c[0]))
    cond = threading.Condition()
    in_flight = [0.0]
    errors, stats = [], [0, 0]
    op_counts = np.zeros(all_ops.shape[0], np.uint64)

    def job(tensors, lists, host, nbytes, before, after):
        try:
            ts = set(tensors)
            op_idx = np.nonzero(np.isin(all_ops[:, 0], np.asarray(tensors)))[0]
            ops = all_ops[op_idx]
            zero = np.zeros(0, np.float32)
            shapes = [s if p in ts else (0, 1) for p, s in enumerate(plan.tensor_shapes)]
            full = [[host[a][p] if p in ts else zero for p in range(plan.n_tensors)] for a in range(3)]
            want = oracle.extract(shapes, plan.shard_numels, ops, *full, consts, with_op_counts=True)
            op_counts[op_idx] = want[3]            # disjoint index sets per job
            assert_lists_equal((lp_g, off_g, val_g), want[:3], plan, lists)
            n = 0
            for i, k in enumerate(lists):
                c, d = int(want[0][k]), int(want[0][k + 1])
                n += d - c
                if before is not None:
                    exp = before[i]
                    exp[want[1][c:d]] = want[2][c:d]          # Eq. 7 as a plain indexed store
                    assert np.array_equal(after[i], exp), f"receiver tensor {plan.shard_names[k]} after apply"
            with cond:
                stats[0] += len(lists)
                stats[1] += n
        except BaseException as e:       # surfaces in the main thread
            with cond:
                errors.append(e)
        finally:
            with cond:
                in_flight[0] -= nbytes
                cond.notify_all()

    with ThreadPoolExecutor(max_workers=threads) as pool:
        for tensors, lists in comps:
            nbytes = 12.0 * sum(plan.numel(p) for p in tensors)
            if shards_before is not None:
                nbytes += 4.0 * sum(plan.shard_numels[k] for k in lists)
            with cond:
                cond.wait_for(lambda: in_flight[0] == 0 or in_flight[0] + nbytes <= budget_bytes or errors)
                if errors:
                    break
                in_flight[0] += nbytes
            host = [{p: lst[p].cpu().numpy() for p in tensors} for lst in (st.theta, st.m, st.v)]
            before = after = None
            if shards_before is not None:
                before = [shards_before[k].cpu().numpy().view(np.uint16) for k in lists]
                after = [shards_after[k].cpu().numpy().view(np.uint16) for k in lists]
            pool.submit(job, tensors, lists, host, nbytes, before, after)
    if errors:
        raise errors[0]
    fed = set(int(o[1]) for o in plan.ops)
    for k in range(plan.n_shards):
        if k not in fed:
            assert lp_g[k] == lp_g[k + 1], f"list {plan.shard_names[k]} has no operation but is not empty"
    assert stats[1] == int(lp_g[-1]), "entries compared vs total"
    return stats[0], stats[1], op_counts
