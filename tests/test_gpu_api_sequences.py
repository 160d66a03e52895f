"""Random sequences of calls on long-lived layouts: the library caches pointer tables, grows its
staging buffer, and shares a layout between the ordinary, the per-group and the fixed-scratch
extract.  Whatever the order - new tensors, a capacity too small and then large enough, another
layout in between, apply onto different shard sets - every result must equal the oracle's."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from gpu_util import assert_lists_equal, oracle_extract
from synth import configs, plans
from synth.tensors import Hyper, Spec

pytestmark = pytest.mark.gpu


def _expected_shards(plan, want, fill):
    lp, off, val = want
    out = []
    for k, n in enumerate(plan.shard_numels):
        e = np.full(n, fill, np.uint16)
        seg = slice(int(lp[k]), int(lp[k + 1]))
        e[off[seg]] = val[seg]
        out.append(e)
    return out


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_random_call_sequences(seed):
    rng = np.random.default_rng(seed)
    plan_a = plans.qwen3_dense_plan(1, 2, True, configs.SMALL_DENSE)
    plan_b = plans.random_plan(1020 + seed)
    layouts = {"a": (plan_a, dte.Layout.from_plan(plan_a, 0)), "b": (plan_b, dte.Layout.from_plan(plan_b, 0))}
    states, wants = {}, {}

    def state(key, which, hp):
        k = (key, which, hp.step, hp.lr, hp.wd)
        if k not in states:
            plan = layouts[key][0]
            specs = configs._specs(plan) if key == "a" else [Spec()] * plan.n_tensors
            states[k] = configs.Workload(f"{key}{which}", plan, hp, specs, 900 + which).materialize("cuda")
            wants[k] = oracle_extract(plan, states[k], hp)
        return states[k], wants[k]

    hps = [Hyper(step=100, lr=1e-5, wd=0.01), Hyper(step=7, lr=3e-4, wd=0.1)]
    deltas = {}
    for step in range(28):
        key = "a" if rng.random() < 0.6 else "b"
        plan, lay = layouts[key]
        hp = hps[int(rng.integers(0, 2))]
        st, want = state(key, int(rng.integers(0, 3)), hp)
        total = int(want[0][-1])
        kind = rng.choice(["plain", "small", "static", "groups"])
        tabs = lay.source_tables(st.theta, st.m, st.v)
        if kind == "small" and total > 10:
            d = lay.new_delta(int(rng.integers(1, total)))              # too small: exact sizes, nothing usable
            dte.dte_extract_delta(lay, tabs, *hp.as_args(), d)
            torch.cuda.synchronize()
            assert d.status_bits() & dte.DTE_DEV_OVERFLOW and d.total() == total
            assert np.array_equal(d.list_ptr.cpu().numpy().astype(np.uint64), want[0])
            shard = [torch.full((n,), 3, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
            dte.dte_apply(lay, d, lay.shard_table(shard))               # refused
            torch.cuda.synchronize()
            assert all(bool((s == 3).all()) for s in shard)
            continue
        cap = total + int(rng.integers(0, 5000))
        d = deltas.get((key, cap)) or lay.new_delta(cap)
        deltas[(key, cap)] = d
        if kind == "static" and cap <= 2097152:
            dte.dte_extract_delta_static(lay, tabs, *hp.as_args(), d)
        elif kind == "groups":
            dte.dte_extract_delta_groups(lay, tabs, hp.step, hp.beta1, hp.beta2, hp.eps, [hp.lr], [hp.wd], d)
        else:
            dte.dte_extract_delta(lay, tabs, *hp.as_args(), d)
        torch.cuda.synchronize()
        assert d.status_bits() == 0, (step, kind)
        assert_lists_equal(d.to_host(), want, plan)
        fill = int(rng.integers(1, 32000))
        shards = [torch.full((n,), fill, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
        dte.dte_apply(lay, d, lay.shard_table(shards))
        torch.cuda.synchronize()
        exp = _expected_shards(plan, want, fill)
        for k in range(plan.n_shards):
            assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), exp[k]), (step, kind, plan.shard_names[k])


def test_two_layouts_on_two_streams_and_two_host_threads():
    """Different layouts are independent: two host threads, each with a layout and a stream of its
    own, extract and apply at the same time (the per-device host state of the library - kernel
    attributes, cached tables - is shared between them).  Every result must equal the oracle's."""
    import threading
    cases = []
    for i, plan in enumerate([plans.qwen3_dense_plan(2, 2, True, configs.SMALL_DENSE),
                              plans.qwen3_moe_plan(2, 4, 4, configs.SMALL_MOE)]):
        hp = Hyper(step=50 + i, lr=2e-5, wd=0.01 * i)        # one call with, one without the decay division
        wl = configs.Workload(f"t{i}", plan, hp, configs._specs(plan), 70 + i)
        st = wl.materialize("cuda")
        cases.append((plan, hp, st, oracle_extract(plan, st, hp)))
    errors = []

    def work(plan, hp, st, want):
        try:
            stream = torch.cuda.Stream()
            lay = dte.Layout.from_plan(plan, 0)
            tabs = lay.source_tables(st.theta, st.m, st.v)
            for it in range(20):
                d = lay.new_delta(int(want[0][-1]) + 16 * it)
                shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
                stream.wait_stream(torch.cuda.current_stream())        # the zero fills above
                dte.dte_extract_delta(lay, tabs, *hp.as_args(), d, stream=stream)
                dte.dte_apply(lay, d, lay.shard_table(shards), stream=stream)
                stream.synchronize()
                assert d.status_bits() == 0
                assert_lists_equal(d.to_host(), want, plan)
                exp = _expected_shards(plan, want, 0)
                assert all(np.array_equal(shards[k].cpu().numpy().view(np.uint16), exp[k]) for k in range(plan.n_shards))
        except BaseException as e:
            errors.append(e)

    threads = [threading.Thread(target=work, args=c) for c in cases]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    if errors:
        raise errors[0]
