"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs - bit-exact in the changed set, offsets, values, order and applied shards."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from synth import configs, plans
from synth.tensors import Hyper, Spec
from gpu_util import (assert_lists_equal, expected_shards, initial_shards, oracle_extract,
                      run_extract)

pytestmark = pytest.mark.gpu


def _apply_and_check(plan, st, lay, d, got, want):
    """Apply on the GPU and with the oracle from the same start; compare every shard."""
    start = initial_shards(plan, st)
    bufs = [s.clone() for s in start]
    dte.dte_apply(lay, d, lay.shard_table(bufs))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    host = [s.cpu().numpy().view(np.uint16).copy() for s in start]
    oracle.apply(plan.shard_numels, *want, host)
    for k in range(plan.n_shards):
        assert np.array_equal(bufs[k].cpu().numpy().view(np.uint16), host[k]), plan.shard_names[k]
    # idempotent (Eq. 4 sends target values)
    again = [b.clone() for b in bufs]
    dte.dte_apply(lay, d, lay.shard_table(again))
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(again, bufs))
    return bufs


def _full_parity(wl, capacity=None):
    st = wl.materialize("cuda")
    lay, d = run_extract(wl.plan, st, wl.hp, capacity)
    assert d.status_bits() == 0
    got = d.to_host()
    *want, odd = oracle_extract(wl.plan, st, wl.hp, with_nonfinite=True)
    want = tuple(want)
    assert_lists_equal(got, want, wl.plan)
    cnt = d.counters.cpu().numpy()
    assert cnt[0] == int(want[0][-1]) and cnt[1] == wl.plan.total_scanned_elements()
    assert cnt[3] == odd, "count of non-finite elements"
    bufs = _apply_and_check(wl.plan, st, lay, d, got, want)
    return st, lay, d, got, bufs


def test_config1_single_matrix_tp2():
    wl = configs.config1()
    st, lay, d, got, bufs = _full_parity(wl)
    total = int(got[0][-1])
    assert 0.001 < total / 16777216 < 0.02
    # mirror-association generator: the reconstruction recovers theta_{t-1} almost always,
    # so the receivers end up equal to BF16(theta_t) except for a handful of elements
    want = expected_shards(wl.plan, st)
    stale = sum(int((a != b).sum().item()) for a, b in zip(bufs, want))
    assert stale <= 8


@pytest.mark.parametrize("name", ["dense_tp4", "dense_tp2", "moe", "matrix_tp3_ragged",
                                  "moe_tp8_ep4_replicated_kv", "dense_tp8_replicated_kv"])
def test_small_plans_with_ragged_widths(name):
    plan = {
        "dense_tp4": lambda: plans.qwen3_dense_plan(2, 4, True, configs.SMALL_DENSE),
        "dense_tp2": lambda: plans.qwen3_dense_plan(3, 2, True, configs.SMALL_DENSE),
        "moe": lambda: plans.qwen3_moe_plan(2, 4, 4, configs.SMALL_MOE),
        # receivers above the KV head count (KV heads replicated) and tensor-parallel experts
        "moe_tp8_ep4_replicated_kv": lambda: plans.qwen3_moe_plan(2, 8, 4, configs.SMALL_MOE),
        "dense_tp8_replicated_kv": lambda: plans.qwen3_dense_plan(2, 8, True, dict(configs.SMALL_DENSE, vocab=3008)),
        # 4099 x 1027: nothing is a multiple of 4 -> scalar tiles, ragged tails
        "matrix_tp3_ragged": lambda: plans.single_matrix_plan(3 * 1367, 1027, 3),
    }[name]()
    wl = configs.Workload(name, plan, Hyper(step=100, lr=1e-5, wd=0.01), configs._specs(plan), 21)
    _full_parity(wl)


def test_config2_full_layer_tp4():
    wl = configs.config2()
    st, lay, d, got, bufs = _full_parity(wl, capacity=8_000_000)
    assert lay.num_lists == 32


@pytest.mark.parametrize("point", [(1e-8, 1, 0.1), (1e-6, 100, 0.01), (1e-4, 1, 0.1), (1e-4, 100, 0.01)])
def test_config5_edge_sweep_reduced_dims(point):
    lr, step, wd = point
    wl = configs.config5(lr, step, wd, 1e-3, dims=configs.SMALL_DENSE)
    _full_parity(wl)


def test_config5_nonfinite_robustness():
    wl = configs.config5(1e-4, 1, 0.1, 1e-2, dims=configs.SMALL_DENSE, nonfinite=True)
    st, lay, d, got, bufs = _full_parity(wl)          # compares counters[3] with the oracle's count
    assert int(d.counters[3].item()) >= 20               # the planted NaNs and infinities were seen
    # and the count starts from zero on every call
    run_extract(wl.plan, st, wl.hp, layout=lay, delta=d)
    first = int(d.counters[3].item())
    run_extract(wl.plan, st, wl.hp, layout=lay, delta=d)
    assert int(d.counters[3].item()) == first


def test_row_parallel_non_multiple_of_four_and_single_rows():
    # column splits whose widths are odd, a one-row operation, and an uncovered gap
    p = plans.Plan()
    a = p.add_tensor("a", (37, 1001))
    b = p.add_tensor("b", (5000,))
    k0 = p.add_shard("a.cols", 0, 37 * 333)
    p.add_op(a, k0, (0, 5), (37, 333), 0, 333, (0, 0))
    k1 = p.add_shard("mixed", 1, 9000)
    p.add_op(b, k1, (100, 0), (3000, 1), 0, 1, (10, 0))       # 1-D slice lands at offset 10
    p.add_op(a, k1, (3, 7), (1, 900), 4000, 2000, (0, 50))    # one row, inside a wider row
    k2 = p.add_shard("empty", 2, 0)
    k3 = p.add_shard("untouched", 3, 64)
    k4 = p.add_shard("a.tail", 0, 36 * 1001)
    p.add_op(a, k4, (1, 0), (36, 1001), 0, 1001, (0, 0))
    wl = configs.Workload("odd", p, Hyper(step=3, lr=3e-4, wd=0.1), [Spec(), Spec()], 5)
    st, lay, d, got, bufs = _full_parity(wl)
    lp = got[0]
    assert lp[2] == lp[3] == lp[4]          # empty and untouched lists keep their slot


@pytest.mark.parametrize("rows,block_rows", [(1500, 16), (1500, 8400)])
def test_packed_tiles_next_to_regular_ones(rows, block_rows):
    # thousands of one-row operations (every one a piece of a packed tile) next to two operations
    # made of regular tiles.  With 16 regular tiles the packed launch is the long one and the
    # regular launch, which starts while it runs, finishes first; the gather must still see every
    # record (one gather launch: under 4096 tiles).  With 8400 regular tiles the three-launch
    # gather runs behind both.
    p = plans.Plan()
    a = p.add_tensor("rows", (rows, 700))
    b = p.add_tensor("block", (block_rows, 9216))
    half = block_rows // 2
    k0 = p.add_shard("r0.rows", 0, rows * 350)
    k1 = p.add_shard("r0.block", 0, half * 9216)
    k2 = p.add_shard("r1.rows", 1, rows * 350)
    k3 = p.add_shard("r1.block", 1, half * 9216)
    for r in range(rows):                       # column halves, one row per operation
        p.add_op(a, k0, (r, 0), (1, 350), r * 350, 350, (0, 0))
        p.add_op(a, k2, (r, 350), (1, 350), r * 350, 350, (0, 0))
    p.add_op(b, k1, (0, 0), (half, 9216), 0, 9216, (0, 0))
    p.add_op(b, k3, (half, 0), (half, 9216), 0, 9216, (0, 0))
    wl = configs.Workload("packed", p, Hyper(step=50, lr=2e-5, wd=0.01), [Spec(), Spec()], 13)
    st, lay, d, got, bufs = _full_parity(wl)
    tiles = lay.last_launch()["tiles"]
    assert tiles == block_rows + 2 * ((rows + 7) // 8) and (tiles <= 4096) == (block_rows == 16)
    for _ in range(5):                          # and the same bytes every time
        d2 = lay.new_delta(d.capacity)
        run_extract(p, st, wl.hp, layout=lay, delta=d2)
        assert torch.equal(d2.list_ptr, d.list_ptr)
        assert torch.equal(d2.offsets[:d.total()], d.offsets[:d.total()])


@pytest.mark.parametrize("tiles,packed_tail", [(4032, 0), (4095, 0), (4096, 0), (4095, 1), (4096, 1), (4097, 0), (4160, 0)])
def test_tile_counts_around_the_switch_between_one_gather_launch_and_three(tiles, packed_tail):
    """Up to 4096 placement records (64 gather blocks) the gather is one launch in which every
    block scans all records; beyond, three launches.  Counts just below, at and just above the
    switch, with the last block full and partly filled, and with a packed tile as the last
    record or the one that crosses the limit."""
    p = plans.Plan()
    first = tiles // 2
    a = p.add_tensor("rows", (tiles, 9216))            # one regular tile per row
    k0 = p.add_shard("r0", 0, first * 9216)
    k1 = p.add_shard("r1", 1, (tiles - first) * 9216)
    p.add_op(a, k0, (0, 0), (first, 9216), 0, 9216, (0, 0))
    p.add_op(a, k1, (first, 0), (tiles - first, 9216), 0, 9216, (0, 0))
    specs = [Spec()]
    if packed_tail:
        b = p.add_tensor("tail", (3, 500))             # a short run: one packed tile, the last record
        k2 = p.add_shard("r1.tail", 1, 1500)
        p.add_op(b, k2, (0, 0), (3, 500), 0, 500, (0, 0))
        specs.append(Spec())
    wl = configs.Workload("switch", p, Hyper(step=50, lr=1e-5, wd=0.01), specs, 77)
    st, lay, d, got, bufs = _full_parity(wl)
    info = lay.last_launch()
    n_rec = tiles + packed_tail
    assert info["tiles"] == n_rec
    assert info["kernels"] == (1 if n_rec <= 4096 else 3) + 1 + packed_tail
    assert int(got[0][-1]) > tiles                     # every tile contributes


def test_all_changed_and_none_changed():
    plan = plans.qwen3_dense_plan(1, 4, False, configs.SMALL_DENSE)
    # beta = 0.5, t = 1, m = v = 0.5, eps = 0: u = 1 exactly; lr = 8 moves every element far
    # enough to change its BF16 pattern -> the lists enumerate every receiver slot
    hp = Hyper(step=1, lr=8.0, beta1=0.5, beta2=0.5, eps=0.0, wd=0.0)
    wl = configs.Workload("all", plan, hp, configs._specs(plan), 3)
    st = wl.materialize("cuda")
    st.m = [torch.full_like(x, 0.5) for x in st.m]
    st.v = [torch.full_like(x, 0.5) for x in st.v]
    lay, d = run_extract(plan, st, hp)
    got = d.to_host()
    assert int(got[0][-1]) == plan.total_scanned_elements() and d.status_bits() == 0
    assert_lists_equal(got, oracle_extract(plan, st, hp), plan)
    for k, n in enumerate(plan.shard_numels):
        assert np.array_equal(got[1][int(got[0][k]):int(got[0][k + 1])], np.arange(n, dtype=np.uint32))
    # zero moments (eps > 0): nothing changes
    hp0 = Hyper(step=100, lr=1e-3, wd=0.0)
    st.m = [torch.zeros_like(x) for x in st.m]
    st.v = [torch.zeros_like(x) for x in st.v]
    lay, d = run_extract(plan, st, hp0)
    lp, off, val = d.to_host()
    assert int(lp[-1]) == 0 and np.all(lp == 0) and d.status_bits() == 0
    assert int(oracle_extract(plan, st, hp0)[0][-1]) == 0


def test_capacity_overflow_reports_exact_sizes_and_apply_refuses():
    wl = configs.config2(dims=configs.SMALL_DENSE, hp=Hyper(step=100, lr=1e-4, wd=0.01))
    st = wl.materialize("cuda")
    want = oracle_extract(wl.plan, st, wl.hp)
    total = int(want[0][-1])
    cap = total // 3
    lay, d = run_extract(wl.plan, st, wl.hp, capacity=cap)
    canary = torch.full((16,), 0x5A5A, dtype=torch.int32, device="cuda")
    assert d.status_bits() & dte.DTE_DEV_OVERFLOW
    assert d.total() == total
    assert np.array_equal(d.list_ptr.cpu().numpy().astype(np.uint64), want[0])
    bufs = initial_shards(wl.plan, st)
    before = [b.clone() for b in bufs]
    dte.dte_apply(lay, d, lay.shard_table(bufs))
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(bufs, before))
    # growing the buffers and calling again succeeds
    lay, d = run_extract(wl.plan, st, wl.hp, capacity=total, layout=lay)
    assert d.status_bits() == 0
    assert_lists_equal(d.to_host(), want, wl.plan)
    assert int(canary.sum().item()) == 16 * 0x5A5A


def test_op_counts_right_after_an_overflowing_extract_reads_no_entry():
    # dte_op_counts is meant to be enqueued straight after the extract; when that extract
    # overflowed, list_ptr holds the exact sizes, which point beyond the entry arrays
    wl = configs.config2(dims=configs.SMALL_DENSE, hp=Hyper(step=100, lr=1e-4, wd=0.01))
    st = wl.materialize("cuda")
    lay = dte.Layout.from_plan(wl.plan, 0)
    pool = torch.full((4096 + 64,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    d = lay.new_delta(64)
    # entry arrays carved out of a canary pool: nothing past the 64 entries may be touched
    d.offsets = pool[2048:2048 + 64]
    d.struct.offsets = d.offsets.data_ptr()
    tabs = lay.source_tables(st.theta, st.m, st.v)
    dte.dte_extract_delta(lay, tabs, *wl.hp.as_args(), d)
    counts = dte.dte_op_counts(lay, d)
    torch.cuda.synchronize()
    assert d.status_bits() & dte.DTE_DEV_OVERFLOW and d.total() > 64
    assert int(counts.abs().sum().item()) == 0
    assert bool((pool[:2048] == 0x5A5A5A5A).all()) and bool((pool[2048 + 64:] == 0x5A5A5A5A).all())
    # a complete delta on the same layout gives the real counts again
    d2 = lay.new_delta(d.total())
    dte.dte_extract_delta(lay, tabs, *wl.hp.as_args(), d2)
    counts = dte.dte_op_counts(lay, d2)
    torch.cuda.synchronize()
    assert d2.status_bits() == 0 and int(counts.sum().item()) == d2.total()


def test_apply_flags_out_of_range_offsets():
    plan = plans.single_matrix_plan(64, 64, 2)
    wl = configs.Workload("b", plan, Hyper(step=1, lr=0.5, wd=0.0), configs._specs(plan, Spec(sigma_g=1.0)), 3)
    st = wl.materialize("cuda")
    lay, d = run_extract(plan, st, wl.hp)
    d.offsets[5] = 2048          # == numel of shard 0: out of range
    bufs = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    guard = torch.zeros(4096, dtype=torch.int16, device="cuda")
    dte.dte_apply(lay, d, lay.shard_table(bufs))
    torch.cuda.synchronize()
    assert d.status_bits() & dte.DTE_DEV_BOUNDS
    assert int(guard.abs().sum().item()) == 0


def test_deterministic_bytes_over_repeated_calls():
    wl = configs.config1(rows=2048, cols=4096)
    st = wl.materialize("cuda")
    lay, d = run_extract(wl.plan, st, wl.hp, capacity=1 << 20)
    ref = [x.clone() for x in (d.offsets[:d.total()], d.values[:d.total()], d.list_ptr)]
    for _ in range(10):
        d.offsets.zero_()
        d.values.zero_()
        run_extract(wl.plan, st, wl.hp, layout=lay, delta=d)
        assert torch.equal(d.offsets[:d.total()], ref[0])
        assert torch.equal(d.values[:d.total()], ref[1])
        assert torch.equal(d.list_ptr, ref[2])


def test_host_buffer_variant_matches_device_variant():
    wl = configs.config2(dims=configs.SMALL_DENSE, hp=Hyper(step=100, lr=1e-5, wd=0.01))
    st = wl.materialize("cuda")
    lay, d = run_extract(wl.plan, st, wl.hp)
    want = d.to_host()
    th, mm, vv = ([x.cpu().pin_memory() for x in a] for a in (st.theta, st.m, st.v))
    ws = torch.empty(lay.host_workspace_bytes, dtype=torch.uint8, device="cuda")
    d2 = lay.new_delta(lay.num_elements)
    res = dte.HostResult(lay.num_lists, d2.capacity)
    dte.dte_extract_delta_host(lay, th, mm, vv, *wl.hp.as_args(), ws, d2, res)
    got = res.arrays()
    assert_lists_equal(got, want, wl.plan)
    assert int(res.counters[0]) == int(want[0][-1])
    assert_lists_equal(got, oracle_extract(wl.plan, st, wl.hp), wl.plan)


def test_layout_errors():
    ok_ops = [(0, 0, 0, 0, 8, 8, 0, 8, 0, 0)]
    for shapes, numels, ops in [
        ([(8, 8)], [64], [(0, 0, 0, 0, 9, 8, 0, 8, 0, 0)]),             # leaves the source
        ([(8, 8)], [63], ok_ops),                                         # leaves the shard
        ([(8, 8)], [64], [(0, 0, 0, 0, 8, 4, 0, 8, 0, 0)]),             # partial rows: not contiguous
        ([(8, 8)], [64], [(0, 0, 0, 0, 4, 8, 0, 8, 0, 0), (0, 0, 2, 0, 4, 8, 0, 8, 3, 0)]),  # overlap
        ([(8, 8)], [64], [(1, 0, 0, 0, 8, 8, 0, 8, 0, 0)]),             # unknown tensor
        ([(8, 8)], [1 << 32], ok_ops),                                    # offsets would not fit uint32
    ]:
        with pytest.raises(dte.DteError) as e:
            dte.Layout(shapes, numels, ops)
        assert e.value.status == 2
    lay = dte.Layout([(8, 8)], [64], ok_ops)
    t = torch.zeros(65, dtype=torch.float32, device="cuda")
    with pytest.raises(dte.DteError):                                     # step 0
        dte.dte_extract_delta(lay, lay.source_tables([t[:64]], [t[:64]], [t[:64]]), 0, 1e-3, 0.9, 0.999, 1e-8, 0.0,
                              lay.new_delta(64))


def test_source_tensors_that_are_only_four_byte_aligned():
    # views into flat buffers at odd element offsets (a flat optimizer buffer cut at arbitrary
    # elements): 128-bit loads are not possible, the call falls back to scalar loads and must give
    # the same lists; the next call with aligned tensors goes back to the fast path
    plan = plans.qwen3_dense_plan(1, 4, True, configs.SMALL_DENSE)
    wl = configs.Workload("views", plan, Hyper(step=100, lr=1e-5, wd=0.01), configs._specs(plan), 19)
    st = wl.materialize("cuda")
    want = oracle_extract(plan, st, wl.hp)

    def shifted(lst, k):
        out = []
        for x in lst:
            buf = torch.empty(x.numel() + 4, dtype=torch.float32, device="cuda")
            buf[k:k + x.numel()] = x
            out.append(buf[k:k + x.numel()])
        return out

    lay = dte.Layout.from_plan(plan, 0)
    for k_theta, k_m, k_v in [(1, 2, 3), (3, 0, 0), (0, 0, 1)]:
        th, mm, vv = shifted(st.theta, k_theta), shifted(st.m, k_m), shifted(st.v, k_v)
        assert th[0].data_ptr() % 16 == 4 * k_theta
        d = lay.new_delta(lay.num_elements)
        dte.dte_extract_delta(lay, lay.source_tables(th, mm, vv), *wl.hp.as_args(), d)
        torch.cuda.synchronize()
        assert d.status_bits() == 0
        assert_lists_equal(d.to_host(), want, plan)
    d = lay.new_delta(lay.num_elements)
    dte.dte_extract_delta(lay, lay.source_tables(st.theta, st.m, st.v), *wl.hp.as_args(), d)
    torch.cuda.synchronize()
    assert_lists_equal(d.to_host(), want, plan)


def test_empty_layouts_and_empty_operations():
    # no operations at all: every list empty, nothing launched
    lay = dte.Layout([(8, 8)], [64, 0, 5], [])
    d = lay.new_delta(4)
    t = torch.ones(64, dtype=torch.float32, device="cuda")
    d.list_ptr.fill_(7)
    dte.dte_extract_delta(lay, lay.source_tables([t], [t], [t]), 1, 1e-3, 0.9, 0.999, 1e-8, 0.0, d)
    torch.cuda.synchronize()
    assert d.total() == 0 and d.status_bits() == 0 and int(d.list_ptr.abs().sum()) == 0
    bufs = [torch.zeros(max(1, n), dtype=torch.int16, device="cuda") for n in (64, 0, 5)]
    dte.dte_apply(lay, d, lay.shard_table(bufs))
    torch.cuda.synchronize()
    # an operation with an empty extent is legal and contributes nothing; tensor 1 is unused (NULL)
    lay = dte.Layout([(8, 8), (4, 4)], [64], [(0, 0, 0, 0, 8, 8, 0, 8, 0, 0), (1, 0, 0, 0, 0, 4, 0, 4, 0, 0)])
    d = lay.new_delta(64)
    m = torch.full((64,), 0.5, dtype=torch.float32, device="cuda")
    dte.dte_extract_delta(lay, lay.source_tables([t, None], [m, None], [m, None]), 1, 8.0, 0.5, 0.5, 0.0, 0.0, d)
    torch.cuda.synchronize()
    assert d.total() == 64 and lay.num_elements == 64


def test_offsets_up_to_the_uint32_limit():
    # destination tensor of 2^32 - 1 elements: offsets beyond 2^31 must survive extract and apply
    free, _ = torch.cuda.mem_get_info()
    if free < 12e9:
        pytest.skip("needs 12 GB of device memory")
    numel = (1 << 32) - 1
    rows, cols = 40, 1000
    base = numel - rows * cols                      # the block ends at the very last slot
    plan = plans.Plan()
    a = plan.add_tensor("a", (rows, cols))
    k = plan.add_shard("huge", 0, numel)
    plan.add_op(a, k, (0, 0), (rows, cols), base, cols, (0, 0))
    wl = configs.Workload("huge", plan, Hyper(step=100, lr=1e-4, wd=0.01), [Spec()], 17)
    st = wl.materialize("cuda")
    lay, d = run_extract(plan, st, wl.hp)
    got = d.to_host()
    want = oracle_extract(plan, st, wl.hp)
    assert_lists_equal(got, want, plan)
    assert int(got[1].max()) > (1 << 31) and int(got[0][-1]) > 100
    shard = torch.zeros(numel, dtype=torch.int16, device="cuda")
    dte.dte_apply(lay, d, lay.shard_table([shard]))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    tail = shard[base:].cpu().numpy().view(np.uint16)
    exp = np.zeros(rows * cols, np.uint16)
    exp[(want[1].astype(np.int64) - base)] = want[2]
    assert np.array_equal(tail, exp)
    assert int(shard[:base][-1000000:].abs().sum()) == 0
    del shard
    torch.cuda.empty_cache()


def test_parameter_groups_lr_and_weight_decay_per_group():
    # group 0: weights (lr, wd); group 1: norms (smaller lr, no weight decay); group 2: embeddings
    plan = plans.qwen3_dense_plan(2, 4, True, configs.SMALL_DENSE)
    groups = [1 if "norm" in n else (2 if n in ("embed_tokens", "lm_head") else 0) for n in plan.tensor_names]
    lr, wd = [1e-4, 3e-5, 5e-5], [0.1, 0.0, 0.3]
    step, b1, b2, eps = 50, 0.9, 0.999, 1e-8
    wl = configs.Workload("groups", plan, Hyper(step=step, lr=lr[0], wd=wd[0]), configs._specs(plan), 41)
    st = wl.materialize("cuda")
    lay = dte.Layout.from_plan(plan, 0, tensor_groups=groups)
    assert lay.num_groups == 3
    d = lay.new_delta(lay.num_elements)
    tabs = lay.source_tables(st.theta, st.m, st.v)
    dte.dte_extract_delta_groups(lay, tabs, step, b1, b2, eps, lr, wd, d)
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    consts = np.stack([oracle.derive_constants(step, lr[g], b1, b2, eps, wd[g]) for g in groups])
    host = lambda lst: [x.cpu().numpy() for x in lst]
    want = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), host(st.theta), host(st.m),
                          host(st.v), consts)
    assert_lists_equal(d.to_host(), want, plan)
    # the single-pair call on the same layout applies one pair to every group
    dte.dte_extract_delta(lay, tabs, step, lr[0], b1, b2, eps, wd[0], d)
    torch.cuda.synchronize()
    one = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), host(st.theta), host(st.m),
                         host(st.v), oracle.derive_constants(step, lr[0], b1, b2, eps, wd[0]))
    assert_lists_equal(d.to_host(), one, plan)
    assert int(one[0][-1]) != int(want[0][-1])
    with pytest.raises(dte.DteError):            # fewer pairs than groups
        dte.dte_extract_delta_groups(lay, tabs, step, b1, b2, eps, lr[:2], wd[:2], d)


def test_op_counts_match_oracle_including_zero_length_operations():
    plan = plans.qwen3_moe_plan(2, 4, 4, configs.SMALL_MOE)
    wl = configs.Workload("counts", plan, Hyper(step=100, lr=3e-6, wd=0.01), configs._specs(plan), 23)
    st = wl.materialize("cuda")
    for p in range(0, plan.n_tensors, 7):          # some tensors do not change at all
        st.m[p].zero_()
        st.v[p].zero_()
    lay, d = run_extract(plan, st, wl.hp)
    got = dte.dte_op_counts(lay, d).cpu().numpy().astype(np.uint64)
    c = oracle.derive_constants(*wl.hp.as_args())
    host = lambda lst: [x.cpu().numpy() for x in lst]
    want = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), host(st.theta), host(st.m),
                          host(st.v), c, with_op_counts=True)
    assert_lists_equal(d.to_host(), want[:3], plan)
    assert np.array_equal(got, want[3])
    assert (got == 0).sum() > 10 and int(got.sum()) == d.total()


def test_identity_plan_yields_the_canonical_pairs_of_eq4():
    # Section 4.2.1 / 4.4: with an identity plan the lists are I = nonzero(M), V = vec(W_t)[I]
    # per canonical tensor, checked here against the oracle's Eq. 4 mask tensor by tensor
    dense = plans.qwen3_dense_plan(1, 1, True, configs.SMALL_DENSE)
    plan = plans.canonical_plan(dense.tensor_names, dense.tensor_shapes)
    wl = configs.Workload("canonical", plan, Hyper(step=200, lr=2e-6, wd=0.05), configs._specs(plan), 77)
    st = wl.materialize("cuda")
    lay, d = run_extract(plan, st, wl.hp)
    lp, off, val = d.to_host()
    c = oracle.derive_constants(*wl.hp.as_args())
    for p in range(plan.n_tensors):
        mask, v16 = oracle.changed_mask(st.theta[p].cpu().numpy(), st.m[p].cpu().numpy(), st.v[p].cpu().numpy(), c)
        idx = np.nonzero(mask)[0]
        assert np.array_equal(off[int(lp[p]):int(lp[p + 1])], idx.astype(np.uint32)), plan.tensor_names[p]
        assert np.array_equal(val[int(lp[p]):int(lp[p + 1])], v16[idx])
    assert int(lp[-1]) > 1000
