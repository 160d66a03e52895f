"""dte_extract_delta_static, the extract for callers that cannot allocate device memory
(their framework owns the whole GPU through its own allocator, or they sit in a loop where
cudaMalloc's implicit synchronisation is not acceptable).  Its scratch is a fixed array in
the library instead of buffers the layout allocates, so the only question is whether it
produces the same bytes as dte_extract_delta - here on two calls in a row with different
inputs, the second of which finds the first call's leftovers in the shared array.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

import paper_2608_00455_b200 as dte
from synth import configs
from synth.tensors import Hyper
from gpu_util import assert_lists_equal, oracle_extract

pytestmark = pytest.mark.gpu


def _both(lay, st, hp, capacity):
    tabs = lay.source_tables(st.theta, st.m, st.v)
    ref = lay.new_delta(capacity)
    dte.dte_extract_delta(lay, tabs, *hp.as_args(), ref)
    got = lay.new_delta(capacity)
    got.offsets.fill_(-1)
    got.values.fill_(-1)
    dte.dte_extract_delta_static(lay, tabs, *hp.as_args(), got)
    torch.cuda.synchronize()
    return ref, got


def _assert_same(ref, got):
    assert got.status_bits() == 0 and ref.status_bits() == 0
    assert torch.equal(got.counters, ref.counters)
    assert torch.equal(got.list_ptr, ref.list_ptr)
    n = ref.total()
    assert n > 0
    assert torch.equal(got.offsets[:n], ref.offsets[:n])     # bit-exact, as in the parity tests
    assert torch.equal(got.values[:n], ref.values[:n])


def test_static_scratch_extract_matches_the_allocating_one_twice_in_a_row():
    # first call: dense change set (lr large); second call: other data, sparse change set
    wl1 = configs.config2(dims=configs.SMALL_DENSE, hp=Hyper(step=1, lr=1e-4, wd=0.1), seed=11)
    wl2 = configs.config2(dims=configs.SMALL_DENSE, hp=Hyper(step=100, lr=1e-6, wd=0.01), seed=12)
    lay = dte.Layout.from_plan(wl1.plan, 0)
    cap = lay.num_elements
    assert cap <= dte.binding.STATIC_MAX_CAPACITY
    st1 = wl1.materialize("cuda")
    ref1, got1 = _both(lay, st1, wl1.hp, cap)
    _assert_same(ref1, got1)
    st2 = wl2.materialize("cuda")
    ref2, got2 = _both(lay, st2, wl2.hp, cap)
    _assert_same(ref2, got2)
    assert ref2.total() < ref1.total()
    # and not only equal to the other entry point: equal to the oracle, both times
    assert_lists_equal(got1.to_host(), oracle_extract(wl1.plan, st1, wl1.hp), wl1.plan)
    assert_lists_equal(got2.to_host(), oracle_extract(wl2.plan, st2, wl2.hp), wl2.plan)


def test_static_scratch_extract_on_a_layout_with_thousands_of_tiles():
    # 67 M elements = 7 282 tiles: beyond the one-launch gather, so the fixed array also carries the
    # block sums of the three-launch gather; compared with the allocating call, twice in a row
    from synth import plans
    plan = plans.single_matrix_plan(8192, 8192, 2)
    wl = configs.Workload("wide", plan, Hyper(step=100, lr=1e-6, wd=0.01), configs._specs(plan), 14)
    st = wl.materialize("cuda")
    lay = dte.Layout.from_plan(plan, 0)
    for _ in range(2):
        ref, got = _both(lay, st, wl.hp, 1 << 20)
        _assert_same(ref, got)
    assert lay.last_launch()["tiles"] > 4096 and lay.last_launch()["kernels"] == 5


def test_static_scratch_extract_overflow_and_empty_plan():
    # capacity below the number of changed elements: exact sizes reported, nothing written past
    # the caller's arrays (they sit inside a canary pool), same answer as the allocating call
    wl = configs.config2(dims=configs.SMALL_DENSE, hp=Hyper(step=1, lr=1e-4, wd=0.1), seed=13)
    lay = dte.Layout.from_plan(wl.plan, 0)
    st = wl.materialize("cuda")
    tabs = lay.source_tables(st.theta, st.m, st.v)
    ref = lay.new_delta(lay.num_elements)
    dte.dte_extract_delta(lay, tabs, *wl.hp.as_args(), ref)
    cap = 100
    pool32 = torch.full((4096,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    pool16 = torch.full((4096,), 0x5A5A, dtype=torch.int16, device="cuda")
    got = lay.new_delta(cap)
    got.offsets, got.values = pool32[1024:1024 + cap], pool16[1024:1024 + cap]
    got.struct.offsets, got.struct.values = got.offsets.data_ptr(), got.values.data_ptr()
    dte.dte_extract_delta_static(lay, tabs, *wl.hp.as_args(), got)
    torch.cuda.synchronize()
    assert ref.status_bits() == 0 and ref.total() > cap
    assert got.status_bits() & dte.DTE_DEV_OVERFLOW
    assert got.total() == ref.total() and torch.equal(got.list_ptr, ref.list_ptr)
    assert bool((pool32[:1024] == 0x5A5A5A5A).all()) and bool((pool32[1024 + cap:] == 0x5A5A5A5A).all())
    assert bool((pool16[:1024] == 0x5A5A).all()) and bool((pool16[1024 + cap:] == 0x5A5A).all())
    # a plan without operations: every list empty, counters cleared
    empty = dte.Layout([(8, 8)], [64, 0, 5], [])
    d = empty.new_delta(4)
    d.list_ptr.fill_(7)
    d.counters.fill_(9)
    t = torch.ones(64, dtype=torch.float32, device="cuda")
    dte.dte_extract_delta_static(empty, empty.source_tables([t], [t], [t]), 1, 1e-3, 0.9, 0.999, 1e-8, 0.0, d)
    torch.cuda.synchronize()
    assert d.total() == 0 and d.status_bits() == 0 and int(d.list_ptr.abs().sum()) == 0


def test_static_scratch_extract_rejects_what_does_not_fit():
    wl = configs.config2(dims=configs.SMALL_DENSE)
    lay = dte.Layout.from_plan(wl.plan, 0)
    st = wl.materialize("cuda")
    tabs = lay.source_tables(st.theta, st.m, st.v)
    too_big = lay.new_delta(dte.binding.STATIC_MAX_CAPACITY + 1)
    with pytest.raises(dte.DteError) as e:
        dte.dte_extract_delta_static(lay, tabs, *wl.hp.as_args(), too_big)
    assert e.value.status == 3 and "capacity" in str(e.value)
    # a layout with more tiles than the fixed record array: many one-element operations
    n = dte.binding.STATIC_MAX_TILES + 1
    shapes = [(n, 1)]
    ops = [(0, k, k, 0, 1, 1, 0, 1, 0, 0) for k in range(n)]
    big = dte.Layout(shapes, [1] * n, ops)
    z = torch.zeros(n, dtype=torch.float32, device="cuda")
    with pytest.raises(dte.DteError) as e:
        dte.dte_extract_delta_static(big, big.source_tables([z], [z], [z]), 1, 1e-3, 0.9, 0.999, 1e-8, 0.0,
                                     big.new_delta(16))
    assert e.value.status == 3 and "tiles" in str(e.value)
