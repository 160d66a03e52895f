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
