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


def oracle_extract(plan, st, hp, tensors=None):
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

    return oracle.extract(shapes, plan.shard_numels, ops, host(st.theta), host(st.m), host(st.v), c)


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
