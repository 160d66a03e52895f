"""Full-size parity in the launch configuration bench.py times: the whole Qwen3-8B-shaped state
(config 3, 98 GB), the Qwen3-30B-A3B slice (config 4, 90 GB) and the density / edge grid on one
full-dimension layer (config 5), resident on one GPU.  The oracle checks EVERY list and every
receiver tensor after apply: the state is streamed to the host group by group and spread over the
host threads (see gpu_util.full_oracle_parity); nothing is sampled."""
import gc

import numpy as np
import pytest
import torch

import bench
import oracle
import paper_2608_00455_b200 as dte
from synth import configs
from gpu_util import assert_lists_equal, full_oracle_parity

pytestmark = pytest.mark.gpu


def _free():
    gc.collect()
    torch.cuda.empty_cache()


def _need(gb):
    free, total = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip(f"needs {gb} GB of free device memory, {free / 1e9:.0f} GB available")


def _global_properties(plan, lay, d):
    """list_ptr monotone and consistent with the counters; every list strictly ascending and in range."""
    assert d.status_bits() == 0
    lp = d.list_ptr.cpu().numpy().astype(np.int64)
    cnt = d.counters.cpu().numpy()
    assert lp[0] == 0 and np.all(np.diff(lp) >= 0) and lp[-1] == cnt[0]
    assert cnt[1] == plan.total_scanned_elements() == lay.num_elements
    off = d.offsets[:int(lp[-1])].to(torch.int64) & 0xFFFFFFFF
    dif = off[1:] - off[:-1]
    starts = torch.from_numpy(lp[1:-1]).to(off.device)
    starts = starts[(starts > 0) & (starts < off.numel())]
    ok = dif > 0
    ok[starts - 1] = True                       # list boundaries may go down
    assert bool(ok.all())
    numel = torch.tensor(plan.shard_numels, device=off.device)
    counts = torch.from_numpy(np.diff(lp)).to(off.device)
    bound = torch.repeat_interleave(numel, counts)
    assert bool((off < bound).all())
    return lp


def _sampled_lists_equal(wl, st, d, tensors):
    """Oracle on `tensors` only; compare every list that those tensors fill completely."""
    plan = wl.plan
    shapes, ops, host = bench.oracle_inputs(plan, st, tensors)
    c = oracle.derive_constants(*wl.hp.as_args())
    want = oracle.extract(shapes, plan.shard_numels, ops, *host, c)
    chosen = set(tensors)
    lists = [k for k in sorted(set(int(x) for x in ops[:, 1]))
             if all(int(o[0]) in chosen for o in plan.ops if o[1] == k)]
    assert lists
    got = d.to_host()
    assert_lists_equal(got, want, plan, lists)
    return lists, want


def _apply_end_state(plan, st, lay, d, shards, sample_shards):
    """After apply the sampled receiver tensors equal remapped BF16(theta_t) except for the
    elements the reconstruction missed (mirror generator: none to a handful)."""
    dte.dte_apply(lay, d, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    ops_by_shard = {}
    for o in plan.ops:
        ops_by_shard.setdefault(o[1], []).append(o)
    stale = 0
    for k in sample_shards:
        exp = torch.zeros_like(shards[k])
        for (src, _, a0, a1, e0, e1, base, ld, r0, r1) in ops_by_shard[k]:
            s2 = st.theta[src].reshape(plan.tensor_shapes[src])[a0:a0 + e0, a1:a1 + e1]
            exp.as_strided((e0, e1), (ld, 1), base + r0 * ld + r1).copy_(s2.to(torch.bfloat16).view(torch.int16))
        stale += int((exp != shards[k]).sum().item())
    return stale


def test_config3_full_qwen3_8b_state():
    _need(150)
    wl = configs.config3("cuda")
    plan = wl.plan
    st, shards = bench.materialize_resident(wl, torch.device("cuda", 0), dte)
    lay = dte.Layout.from_plan(plan, 0)
    N = lay.num_elements
    assert N == 8191035392
    d = lay.new_delta(int(N * 0.03))
    # the extract that also delivers every receiver's share (Section 4.3 fused into the gather);
    # `d` itself is filled exactly as by dte_extract_delta
    targets = [dte.PushTarget(lay.num_lists, d.capacity, lay.receiver_num_ops(r), "cuda") for r in range(2)]
    dte.dte_extract_delta_push(lay, lay.source_tables(st.theta, st.m, st.v), *wl.hp.as_args(), d, targets, 500)
    torch.cuda.synchronize()
    lp = _global_properties(plan, lay, d)
    assert 0.01 < lp[-1] / N < 0.02
    # every one of the 580 lists (lm_head, the last tensor with the highest tile indices and
    # source offsets, and all 36 layers included) and every receiver tensor after apply
    after = [s.clone() for s in shards]
    dte.dte_apply(lay, d, lay.shard_table(after))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    n_lists, n_entries, op_counts = full_oracle_parity(wl, st, d, shards, after)
    assert n_lists == 580 and n_entries == int(lp[-1])
    del after
    _free()
    _receivers_hold_their_share(plan, lay, d, targets, op_counts, 500)
    del targets
    _free()
    # the storage-path leg below also needs complete oracle lists of a few tensors
    names = plan.tensor_names
    sample = [p for p, n in enumerate(names) if n.startswith("layers.35.")] + [names.index("lm_head")]
    lists, want = _sampled_lists_equal(wl, st, d, sample)
    assert len(lists) == 18
    assert _apply_end_state(plan, st, lay, d, shards, lists) <= 8
    del shards
    _free()
    _storage_path_at_full_size(wl, st, lay, d, lists, want)
    del st, d, lay
    _free()


def _receivers_hold_their_share(plan, lay, d, targets, op_counts, epoch):
    """What the push delivered: every receiver's slice of the (oracle-checked) lists, its list
    boundaries relative to the slice, the oracle's per-operation counts in plan order, the status."""
    lp = d.list_ptr.cpu().numpy().astype(np.int64)
    recv = np.asarray(plan.shard_receivers)
    op_recv = recv[plan.ops_array()[:, 1]]
    for r, t in enumerate(targets):
        mine = np.nonzero(recv == r)[0]
        a, b = int(lp[mine[0]]), int(lp[mine[-1] + 1])
        assert t.status.cpu().tolist() == [b - a, epoch, 0, lay.receiver_num_ops(r)]
        assert torch.equal(t.offsets[:b - a], d.offsets[a:b]) and torch.equal(t.values[:b - a], d.values[a:b])
        want_lp = np.clip(lp, a, b) - a
        assert np.array_equal(t.list_ptr.cpu().numpy(), want_lp)
        mask = op_recv == r
        assert int(mask.sum()) == lay.receiver_num_ops(r)
        assert np.array_equal(t.op_counts[:int(mask.sum())].cpu().numpy().astype(np.uint64), op_counts[mask])
        assert int(op_counts[mask].sum()) == b - a


def _storage_path_at_full_size(wl, st, lay, d, lists, want):
    """Canonical extract -> chunks -> verified read-back -> destination-side mapping, whole state;
    the sampled receiver tensors must hold exactly the oracle's lists scattered into zeros."""
    from synth import plans
    plan = wl.plan
    ident = plans.canonical_plan(plan.tensor_names, plan.tensor_shapes)
    lay_c = dte.Layout.from_plan(ident, 0)
    d_c = lay_c.new_delta(d.capacity)
    dte.dte_extract_delta(lay_c, lay_c.source_tables(st.theta, st.m, st.v), *wl.hp.as_args(), d_c)
    torch.cuda.synchronize()
    assert d_c.status_bits() == 0
    M = d_c.total()
    assert abs(M - d.total()) < 100_000          # only the replicated norms differ
    fmt = dte.DTE_CHUNK_DELTA_PLANES
    cs = dte.ChunkStream(lay_c.num_lists, M, 16384, fmt, lay_c.device)
    dte.dte_pack_chunks(lay_c, d_c, cs)
    n_chunks, nbytes, bits, entries = (int(x) for x in cs.info.cpu().tolist())
    assert bits == 0 and entries == M and n_chunks >= M // 16384
    # sampled chunks against the oracle's writer: the first chunks of the stream (tensor 0), from
    # the oracle's own canonical list of that tensor
    shapes, ops0, host = bench.oracle_inputs(ident, st, [0])
    c = oracle.derive_constants(*wl.hp.as_args())
    o_lp, o_off, o_val = oracle.extract(shapes, ident.shard_numels, ops0, *host, c)
    n0 = int(o_lp[1])
    assert n0 == int(d_c.list_ptr[1].item()) and n0 > 100_000
    o_stream, o_dir = oracle.pack_chunks(o_lp[:2], o_off[:n0], o_val[:n0], 16384, fmt)
    assert np.array_equal(cs.stream[:o_stream.size].cpu().numpy(), o_stream)
    back = lay_c.new_delta(M)
    back.list_ptr.copy_(d_c.list_ptr)
    dte.dte_unpack_chunks(lay_c, cs.stream, cs.directory, n_chunks, back, nbytes=nbytes)
    torch.cuda.synchronize()
    assert back.counters.cpu().tolist() == [M, n_chunks, 0, 0]
    assert torch.equal(back.offsets[:M], d_c.offsets[:M]) and torch.equal(back.values[:M], d_c.values[:M])
    shards2 = [torch.zeros(n, dtype=torch.int16, device="cuda") if k in lists else None
               for k, n in enumerate(plan.shard_numels)]
    dte.dte_apply_canonical(lay, back, lay.shard_table(shards2))
    torch.cuda.synchronize()
    assert back.status_bits() == 0
    w_lp, w_off, w_val = want
    for k in lists:
        exp = np.zeros(plan.shard_numels[k], np.uint16)
        seg = slice(int(w_lp[k]), int(w_lp[k + 1]))
        exp[w_off[seg]] = w_val[seg]
        assert np.array_equal(shards2[k].cpu().numpy().view(np.uint16), exp), plan.shard_names[k]


def test_config4_qwen3_30b_a3b_slice():
    _need(150)
    wl = configs.config4("cuda")
    plan = wl.plan
    assert (plan.n_shards, len(plan.ops)) == (432, 5040)
    st, shards = bench.materialize_resident(wl, torch.device("cuda", 0), dte)
    lay = dte.Layout.from_plan(plan, 0)
    N = lay.num_elements
    d = lay.new_delta(int(N * 0.04))
    dte.dte_extract_delta(lay, lay.source_tables(st.theta, st.m, st.v), *wl.hp.as_args(), d)
    torch.cuda.synchronize()
    _global_properties(plan, lay, d)
    assert wl.notes["cold_experts"] > 0
    # every one of the 432 lists (all 12 layers: attention, router, norms, 128 experts each, cold
    # ones included) and every receiver tensor after apply
    after = [s.clone() for s in shards]
    dte.dte_apply(lay, d, lay.shard_table(after))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    n_lists, n_entries, op_counts = full_oracle_parity(wl, st, d, shards, after)
    assert n_lists == 432 and n_entries == d.total()
    # cold experts (zero state) contribute nothing
    cold = [p for p, n in enumerate(plan.tensor_names) if "experts" in n and wl.specs[p].scale == 0.0]
    assert cold
    for p in cold[:6]:
        assert float(st.m[p].abs().max()) == 0.0 and float(st.v[p].abs().max()) == 0.0
    stale = sum(int((a != b).sum().item()) for a, b in zip(after, _expected(plan, st)))
    assert stale <= 16
    del st, shards, after, d, lay
    _free()


def _expected(plan, st):
    """Remapped BF16(theta_t) of every receiver tensor, one at a time (generator)."""
    ops_by_shard = {}
    for o in plan.ops:
        ops_by_shard.setdefault(o[1], []).append(o)
    for k, n in enumerate(plan.shard_numels):
        exp = torch.zeros(n, dtype=torch.int16, device="cuda")
        for (src, _, a0, a1, e0, e1, base, ld, r0, r1) in ops_by_shard.get(k, []):
            s2 = st.theta[src].reshape(plan.tensor_shapes[src])[a0:a0 + e0, a1:a1 + e1]
            exp.as_strided((e0, e1), (ld, 1), base + r0 * ld + r1).copy_(s2.to(torch.bfloat16).view(torch.int16))
        yield exp


@pytest.mark.parametrize("point", configs.config5_points(), ids=lambda p: f"lr{p[0]:g}-t{p[1]}-wd{p[2]:g}-sg{p[3]:g}")
def test_config5_density_and_edge_grid_full_dimensions(point):
    """The whole grid lr x t x wd (plus the sigma_g = 1e-2 point) on the full-dimension Qwen3-8B
    layer with planted ties, zeros, extremes and subnormals: every list and every receiver tensor
    against the oracle."""
    _need(12)
    lr, step, wd, sigma_g = point
    wl = configs.config5(lr, step, wd, sigma_g)
    plan = wl.plan
    st = wl.materialize("cuda")
    lay = dte.Layout.from_plan(plan, 0)
    assert lay.num_elements == 192971776
    d = lay.new_delta(lay.num_elements // 2 + 4096)
    dte.dte_extract_delta(lay, lay.source_tables(st.theta, st.m, st.v), *wl.hp.as_args(), d)
    torch.cuda.synchronize()
    _global_properties(plan, lay, d)
    from gpu_util import initial_shards
    before = initial_shards(plan, st)
    after = [s.clone() for s in before]
    dte.dte_apply(lay, d, lay.shard_table(after))
    torch.cuda.synchronize()
    assert d.status_bits() == 0
    n_lists, n_entries, op_counts = full_oracle_parity(wl, st, d, before, after)
    assert n_lists == 32 and n_entries == d.total()
    del st, before, after, d, lay
    _free()
