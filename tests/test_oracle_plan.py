"""Pins for the oracle's remap (Eq. 5-6), list order and apply (Eq. 7), and for
the plan builders themselves, against tensor slicing and invariants."""
import numpy as np
import pytest
import torch

import oracle
from synth import configs, plans
from synth.tensors import Hyper


def _all_changed_state(plan, seed=0):
    """theta/m/v for which every element's BF16 pattern changes: lr is huge, u = 1."""
    rng = np.random.default_rng(seed)
    th, mm, vv = [], [], []
    for p in range(plan.n_tensors):
        n = plan.numel(p)
        th.append((rng.standard_normal(n) * 0.02).astype(np.float32))
        mm.append(np.full(n, 0.5, np.float32))
        vv.append(np.full(n, 0.5, np.float32))
    # beta=0.5, t=1: m/0.5 = 1, v/0.5 = 1, sqrt = 1, eps = 0 -> u = 1; prev = theta + 8
    c = oracle.derive_constants(1, 8.0, 0.5, 0.5, 0.0, 0.0)
    return th, mm, vv, c


def _bf16_bits_t(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(x).to(torch.bfloat16).view(torch.int16)


SMALL_PLANS = {
    "matrix_tp1": lambda: plans.single_matrix_plan(24, 20, 1),
    "matrix_tp2": lambda: plans.single_matrix_plan(24, 20, 2),
    "dense_tp4": lambda: plans.qwen3_dense_plan(2, 4, True, configs.SMALL_DENSE),
    "dense_tp2": lambda: plans.qwen3_dense_plan(1, 2, True, configs.SMALL_DENSE),
    "moe": lambda: plans.qwen3_moe_plan(2, 4, 4, configs.SMALL_MOE),
    "moe_tp8_ep4_replicated_kv": lambda: plans.qwen3_moe_plan(1, 8, 4, configs.SMALL_MOE),
    "dense_tp8_replicated_kv": lambda: plans.qwen3_dense_plan(1, 8, False, configs.SMALL_DENSE),
}


@pytest.mark.parametrize("name", list(SMALL_PLANS))
def test_coverage_each_slot_once_and_reassembly(name):
    plan = SMALL_PLANS[name]()
    th, mm, vv, c = _all_changed_state(plan)
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(),
                                  th, mm, vv, c)
    # every receiver slot is produced exactly once, in ascending order, lists in shard order
    for k, n in enumerate(plan.shard_numels):
        seg = off[int(lp[k]):int(lp[k + 1])]
        assert np.array_equal(seg, np.arange(n, dtype=np.uint32)), plan.shard_names[k]
    assert int(lp[-1]) == sum(plan.shard_numels) == plan.total_scanned_elements()
    # values: the lists are exactly the dense BF16 tensors pushed through strided slicing
    shards = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, [_bf16_bits_t(t) for t in th], shards)
    want = torch.cat(shards).numpy().view(np.uint16)
    assert np.array_equal(val, want)


@pytest.mark.parametrize("seed", range(12))
def test_random_plans_remap_like_strided_slicing(seed):
    # arbitrary hyper-rectangles with gaps and replication: with every element changed, list k is
    # exactly the covered slots of shard k in ascending order, carrying the sliced dense values
    plan = plans.random_plan(1000 + seed)
    th, mm, vv, c = _all_changed_state(plan, seed)
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    marker = -1                                         # 0xFFFF cannot come out of these values
    shards = [torch.full((n,), marker, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, [_bf16_bits_t(t).reshape(plan.tensor_shapes[i]) for i, t in enumerate(th)], shards)
    assert int(lp[-1]) == plan.total_scanned_elements()
    for k, buf in enumerate(shards):
        b = buf.numpy().view(np.uint16)
        covered = np.nonzero(b != 0xFFFF)[0]
        seg = slice(int(lp[k]), int(lp[k + 1]))
        assert np.array_equal(off[seg], covered.astype(np.uint32)), plan.shard_names[k]
        assert np.array_equal(val[seg], b[covered])


def test_tp1_is_identity_and_row_split_is_an_offset():
    plan = plans.single_matrix_plan(24, 20, 1)
    th, mm, vv, c = _all_changed_state(plan)
    lp, off, _ = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    assert np.array_equal(off, np.arange(24 * 20, dtype=np.uint32))          # j = i
    plan = plans.single_matrix_plan(24, 20, 3)
    # change only a few chosen source indices
    th, mm, vv, c = _all_changed_state(plan)
    mm[0][:] = 0.0
    vv[0][:] = 0.0
    c = oracle.derive_constants(1, 8.0, 0.5, 0.5, 1.0, 0.0)      # eps = 1: m = 0 -> u = 0 -> unchanged
    chosen = np.array([0, 19, 20, 159, 160, 161, 319, 320, 479])
    mm[0][chosen] = 0.5
    vv[0][chosen] = 0.5
    lp, off, _ = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    rows_r = 8
    got = [(r, int(j)) for r in range(3) for j in off[int(lp[r]):int(lp[r + 1])]]
    want = [(int(i) // (rows_r * 20), int(i) - (int(i) // (rows_r * 20)) * rows_r * 20) for i in chosen]
    assert got == want


def _textbook_layer_shards(dense, dims, R):
    """Receiver tensors of one dense layer from torch.chunk / torch.cat (the usual TP rules)."""
    out = []
    for r in range(R):
        q, k, v = (dense[n].chunk(R, 0)[r] for n in ("q", "k", "v"))
        out.append(torch.cat([q, k, v], 0))
        out.append(dense["o"].chunk(R, 1)[r])
        out.append(torch.cat([dense["gate"].chunk(R, 0)[r], dense["up"].chunk(R, 0)[r]], 0))
        out.append(dense["down"].chunk(R, 1)[r])
        out += [dense[n] for n in ("q_norm", "k_norm", "ln1", "ln2")]
    return out


@pytest.mark.parametrize("R", [1, 2, 4])
def test_dense_layer_plan_equals_textbook_tp_sharding(R):
    d = configs.SMALL_DENSE
    plan = plans.qwen3_dense_plan(1, R, False, d)
    order = ["q", "k", "v", "o", "gate", "up", "down", "q_norm", "k_norm", "ln1", "ln2"]
    g = torch.Generator().manual_seed(1)
    dense = {}
    for p, key in enumerate(order):
        shp = plan.tensor_shapes[p]
        t = torch.randint(-30000, 30000, shp, generator=g, dtype=torch.int16)
        dense[key] = t if "norm" not in key and not key.startswith("ln") else t.reshape(-1)
    shards = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, [dense[k] for k in order], shards)
    want = _textbook_layer_shards(dense, d, R)
    assert len(want) == plan.n_shards
    for k, w in enumerate(want):
        assert torch.equal(shards[k], w.reshape(-1)), plan.shard_names[k]
    # App. B shapes (Eq. 12): fused qkv rows = (h_q + 2 h_kv) d_h / R
    assert plan.shard_numels[0] == (d["q_heads"] + 2 * d["kv_heads"]) * d["head_dim"] // R * d["hidden"]


def test_moe_plan_equals_stacked_experts():
    d = configs.SMALL_MOE
    plan = plans.qwen3_moe_plan(1, 4, 4, d)
    g = torch.Generator().manual_seed(2)
    dense = [torch.randint(-30000, 30000, s, generator=g, dtype=torch.int16) for s in plan.tensor_shapes]
    shards = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, dense, shards)
    name_to_p = {n: i for i, n in enumerate(plan.tensor_names)}
    e_loc = d["experts"] // 4
    for r in range(4):
        w13 = torch.stack([torch.cat([dense[name_to_p[f"layers.0.experts.{e}.gate_proj"]],
                                      dense[name_to_p[f"layers.0.experts.{e}.up_proj"]]], 0)
                           for e in range(r * e_loc, (r + 1) * e_loc)])
        w2 = torch.stack([dense[name_to_p[f"layers.0.experts.{e}.down_proj"]]
                          for e in range(r * e_loc, (r + 1) * e_loc)])
        k13 = plan.shard_names.index(f"r{r}.layers.0.w13")
        k2 = plan.shard_names.index(f"r{r}.layers.0.w2")
        assert torch.equal(shards[k13], w13.reshape(-1))
        assert torch.equal(shards[k2], w2.reshape(-1))
        kr = plan.shard_names.index(f"r{r}.layers.0.router")
        assert torch.equal(shards[kr], dense[name_to_p["layers.0.router"]].reshape(-1))


def test_replicated_kv_heads_and_expert_tensor_parallelism_equal_textbook_sharding():
    # receivers above the KV head count hold one whole KV head each (head r // replicas), and an
    # expert-parallel group of tp/ep ranks splits its experts: gate/up by rows, down by columns
    d = configs.SMALL_MOE                               # 8 Q heads, 4 KV heads, 16 experts
    tp, ep = 8, 4
    etp, hd, hkv = tp // ep, d["head_dim"], d["kv_heads"]
    plan = plans.qwen3_moe_plan(1, tp, ep, d)
    g = torch.Generator().manual_seed(3)
    dense = [torch.randint(-30000, 30000, s, generator=g, dtype=torch.int16) for s in plan.tensor_shapes]
    shards = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, dense, shards)
    at = {n: dense[i] for i, n in enumerate(plan.tensor_names)}
    e_loc = d["experts"] // ep
    for r in range(tp):
        q = at["layers.0.q_proj"].chunk(tp, 0)[r]
        j = r // (tp // hkv)
        k = at["layers.0.k_proj"].view(hkv, hd, -1)[j]
        v = at["layers.0.v_proj"].view(hkv, hd, -1)[j]
        got = shards[plan.shard_names.index(f"r{r}.layers.0.qkv_proj")]
        assert torch.equal(got, torch.cat([q, k, v], 0).reshape(-1))
        experts = range((r // etp) * e_loc, (r // etp + 1) * e_loc)
        w13 = torch.stack([torch.cat([at[f"layers.0.experts.{e}.gate_proj"].chunk(etp, 0)[r % etp],
                                      at[f"layers.0.experts.{e}.up_proj"].chunk(etp, 0)[r % etp]], 0) for e in experts])
        w2 = torch.stack([at[f"layers.0.experts.{e}.down_proj"].chunk(etp, 1)[r % etp] for e in experts])
        assert torch.equal(shards[plan.shard_names.index(f"r{r}.layers.0.w13")], w13.reshape(-1))
        assert torch.equal(shards[plan.shard_names.index(f"r{r}.layers.0.w2")], w2.reshape(-1))
    # the dense model the same way: Qwen3-8B-like heads at TP 8 with 4 KV heads
    dd = configs.SMALL_DENSE
    dp = plans.qwen3_dense_plan(1, 8, False, dd)
    dense = [torch.randint(-30000, 30000, s, generator=g, dtype=torch.int16) for s in dp.tensor_shapes]
    shards = [torch.zeros(n, dtype=torch.int16) for n in dp.shard_numels]
    plans.scatter_dense(dp, dense, shards)
    for r in range(8):
        want = torch.cat([dense[0].chunk(8, 0)[r], dense[1].view(4, dd["head_dim"], -1)[r // 2],
                          dense[2].view(4, dd["head_dim"], -1)[r // 2]], 0)
        assert torch.equal(shards[dp.shard_names.index(f"r{r}.layers.0.qkv_proj")], want.reshape(-1))


def test_plan_counts_match_the_full_size_models():
    p2 = plans.qwen3_dense_plan(1, 4, False)
    assert (p2.n_shards, len(p2.ops)) == (32, 44)
    assert p2.total_source_elements() == 192946432
    assert p2.total_scanned_elements() == 192946432 + 3 * 8448     # norms replicated 4x
    p4 = plans.qwen3_moe_plan(1, 4, 4)
    assert (p4.n_shards, len(p4.ops)) == (36, 420)
    assert p4.total_source_elements() == 623120640
    assert p4.total_scanned_elements() == 623120640 + 3 * 266496
    assert max(p4.shard_numels) < 2 ** 32


def _random_sparse_case(plan, seed, lr=1e-5):
    wl = configs.Workload("t", plan, Hyper(step=100, lr=lr, wd=0.01),
                          configs._specs(plan), seed)
    st = wl.materialize("cpu")
    c = oracle.derive_constants(*wl.hp.as_args())
    th, mm, vv = ([x.numpy() for x in a] for a in (st.theta, st.m, st.v))
    return wl, st, c, th, mm, vv


@pytest.mark.parametrize("name", ["dense_tp4", "moe"])
def test_lists_sorted_unique_and_consistent_with_mask(name):
    plan = SMALL_PLANS[name]()
    wl, st, c, th, mm, vv = _random_sparse_case(plan, 3)
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    assert lp[0] == 0 and np.all(np.diff(lp.astype(np.int64)) >= 0)
    for k in range(plan.n_shards):
        seg = off[int(lp[k]):int(lp[k + 1])].astype(np.int64)
        assert np.all(np.diff(seg) > 0)
        assert seg.size == 0 or seg[-1] < plan.shard_numels[k]
    # dense route: mark changed elements per source tensor, push the marks and the BF16
    # values through strided slicing, read the lists off the shards with nonzero()
    marks, vals = [], []
    for p in range(plan.n_tensors):
        mk, v16 = oracle.changed_mask(th[p], mm[p], vv[p], c)
        marks.append(torch.from_numpy(mk.astype(np.int16)))
        vals.append(torch.from_numpy(v16.view(np.int16).copy()))
    mk_sh = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    v_sh = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, marks, mk_sh)
    plans.scatter_dense(plan, vals, v_sh)
    for k in range(plan.n_shards):
        idx = torch.nonzero(mk_sh[k]).reshape(-1)
        assert np.array_equal(off[int(lp[k]):int(lp[k + 1])], idx.numpy().astype(np.uint32))
        assert np.array_equal(val[int(lp[k]):int(lp[k + 1])].view(np.int16), v_sh[k][idx].numpy())
    assert 0 < int(lp[-1]) < sum(plan.shard_numels) // 4


def test_apply_idempotent_untouched_and_end_state():
    plan = SMALL_PLANS["dense_tp4"]()
    wl, st, c, th, mm, vv = _random_sparse_case(plan, 4)
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    # receiver starts from BF16(reconstruction); after apply it must equal BF16(theta_t) everywhere
    prev16 = [torch.from_numpy(oracle.bf16_rne(oracle.invert(th[p], mm[p], vv[p], c)).view(np.int16).copy())
              for p in range(plan.n_tensors)]
    cur16 = [_bf16_bits_t(th[p]) for p in range(plan.n_tensors)]
    start = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    want = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, prev16, start)
    plans.scatter_dense(plan, cur16, want)
    bufs = [s.numpy().view(np.uint16).copy() for s in start]
    oracle.apply(plan.shard_numels, lp, off, val, bufs)
    for k in range(plan.n_shards):
        assert np.array_equal(bufs[k], want[k].numpy().view(np.uint16)), plan.shard_names[k]
        # positions not listed keep their old contents
        keep = np.ones(plan.shard_numels[k], bool)
        keep[off[int(lp[k]):int(lp[k + 1])]] = False
        assert np.array_equal(bufs[k][keep], start[k].numpy().view(np.uint16)[keep])
    again = [b.copy() for b in bufs]
    oracle.apply(plan.shard_numels, lp, off, val, again)
    assert all(np.array_equal(a, b) for a, b in zip(again, bufs))
    # out-of-range index is refused
    bad = off.copy()
    bad[0] = plan.shard_numels[0]
    with pytest.raises(ValueError):
        oracle.apply(plan.shard_numels, lp, bad, val, [b.copy() for b in bufs])


@pytest.mark.parametrize("variant", ["mirror", "trainer"])
def test_stale_elements_after_apply_equal_false_negatives(variant):
    # receiver starts from BF16(true theta_{t-1}); elements still wrong after apply are exactly
    # those that truly changed but were not emitted (reconstruction missed them)
    plan = plans.single_matrix_plan(512, 2048, 2)
    wl = configs.Workload("t", plan, Hyper(step=100, lr=1e-5, wd=0.1), configs._specs(plan), 9,
                          variant=variant)
    st = wl.materialize("cpu")
    c = oracle.derive_constants(*wl.hp.as_args())
    th, mm, vv = ([x.numpy() for x in a] for a in (st.theta, st.m, st.v))
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    start = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    want = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, [st.prev_bf16[0].view(torch.int16)], start)
    plans.scatter_dense(plan, [_bf16_bits_t(th[0])], want)
    bufs = [s.numpy().view(np.uint16).copy() for s in start]
    oracle.apply(plan.shard_numels, lp, off, val, bufs)
    stale = sum(int((b != w.numpy().view(np.uint16)).sum()) for b, w in zip(bufs, want))
    emitted, _ = oracle.changed_mask(th[0], mm[0], vv[0], c)
    truly = (st.prev_bf16[0].view(torch.int16) != _bf16_bits_t(th[0])).numpy()
    fn = int((truly & ~emitted.astype(bool)).sum())
    assert stale == fn
    if variant == "mirror":
        assert fn <= 2          # the mirror association is recovered almost always exactly
    assert emitted.sum() > 1000


def test_plan_errors_are_reported():
    plan = plans.single_matrix_plan(8, 8, 2)
    th, mm, vv, c = _all_changed_state(plan)
    ops = plan.ops_array().copy()
    ops[1, 8] = 0          # both operations now write rows 0..3 of ... different shards: fine
    ops[1, 1] = 0          # same shard, same rows -> duplicate slots
    with pytest.raises(ValueError):
        oracle.extract(plan.tensor_shapes, plan.shard_numels, ops, th, mm, vv, c)
    ops = plan.ops_array().copy()
    ops[0, 6] = 40         # pushes the block past the end of the shard
    with pytest.raises(ValueError):
        oracle.extract(plan.tensor_shapes, plan.shard_numels, ops, th, mm, vv, c)


def test_per_tensor_constants_equal_one_tensor_at_a_time():
    """Parameter groups (Section 4.1: lambda and eta_t belong to the element's group): the
    extract with one row of constants per tensor equals separate single-group extracts of
    each tensor's operations, list by list."""
    plan = plans.qwen3_dense_plan(1, 2, False, configs.SMALL_DENSE)
    wl, st, _, th, mm, vv = _random_sparse_case(plan, 6, lr=1e-4)
    rows = []
    for p, name in enumerate(plan.tensor_names):
        norm = "norm" in name
        rows.append(oracle.derive_constants(100, 3e-5 if norm else 1e-4, 0.9, 0.999, 1e-8, 0.0 if norm else 0.1))
    consts = np.stack(rows)
    assert consts[0, 2] != 1.0 and consts[-1, 2] == 1.0
    lp, off, val = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, consts)
    merged = [[] for _ in range(plan.n_shards)]
    ops = plan.ops_array()
    for p in range(plan.n_tensors):
        sub = ops[ops[:, 0] == p]
        l1, o1, v1 = oracle.extract(plan.tensor_shapes, plan.shard_numels, sub, th, mm, vv, consts[p])
        for k in range(plan.n_shards):
            merged[k] += list(zip(o1[int(l1[k]):int(l1[k + 1])], v1[int(l1[k]):int(l1[k + 1])]))
    for k in range(plan.n_shards):
        got = list(zip(off[int(lp[k]):int(lp[k + 1])], val[int(lp[k]):int(lp[k + 1])]))
        assert got == sorted(merged[k])
    assert int(lp[-1]) > 1000


def test_op_counts_keep_every_planned_operation():
    """c_o = |I_o| per operation in plan order, zero-length ones included (Section 4.3): they add
    up to the list lengths and equal a brute-force count of the list entries that fall into each
    operation's destination block."""
    plan = plans.qwen3_moe_plan(1, 4, 4, configs.SMALL_MOE)
    wl, st, c, th, mm, vv = _random_sparse_case(plan, 8, lr=3e-6)
    ops = plan.ops_array().copy()
    ops = np.concatenate([ops, [[0, 0, 0, 0, 0, ops[0, 5], 0, ops[0, 7], 0, 0]]])   # an empty overlap
    lp, off, val, cnt = oracle.extract(plan.tensor_shapes, plan.shard_numels, ops, th, mm, vv, c,
                                       with_op_counts=True)
    assert cnt.shape == (ops.shape[0],) and cnt[-1] == 0 and (cnt == 0).sum() > 1
    for k in range(plan.n_shards):
        assert int(cnt[ops[:, 1] == k].sum()) == int(lp[k + 1] - lp[k])
    for o, (src, dst, a0, a1, e0, e1, base, ld, r0, r1) in enumerate(ops):
        begin = base + r0 * ld + r1
        end = begin + e0 * e1          # whole destination rows: a contiguous block
        seg = off[int(lp[dst]):int(lp[dst + 1])].astype(np.int64)
        assert int(((seg >= begin) & (seg < end)).sum()) == int(cnt[o])


# ---------------------------------------------------------------- destination-side mapping (Section 4.4)

def _canonical_lists(plan, th, mm, vv, c):
    ident = plans.canonical_plan(plan.tensor_names, plan.tensor_shapes)
    return oracle.extract(ident.tensor_shapes, ident.shard_numels, ident.ops_array(), th, mm, vv, c)


@pytest.mark.parametrize("name", list(SMALL_PLANS) + [f"random{i}" for i in range(6)])
def test_canonical_entries_mapped_at_the_destination_equal_dense_slicing(name):
    plan = plans.random_plan(1000 + int(name[6:])) if name.startswith("random") else SMALL_PLANS[name]()
    hp = Hyper(step=50, lr=3e-5, wd=0.01)
    wl = configs.Workload(name, plan, hp, configs._specs(plan), 11)
    st = wl.materialize("cpu")
    th, mm, vv = ([t.numpy() for t in x] for x in (st.theta, st.m, st.v))
    c = oracle.derive_constants(*hp.as_args())
    lp, idx, val = _canonical_lists(plan, th, mm, vv, c)
    assert 0 < int(lp[-1]) < plan.total_source_elements()
    canary = 0x5A5A
    got = [np.full(n, canary, np.uint16) for n in plan.shard_numels]
    oracle.apply_canonical(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), lp, idx, val, got)
    # independent statement: a dense tensor holding the target value at changed positions and a
    # marker elsewhere, pushed through strided slicing; marker slots keep the canary
    marker = 0xFFFF
    dense = []
    for p in range(plan.n_tensors):
        d = np.full(plan.numel(p), marker, np.uint16)
        seg = slice(int(lp[p]), int(lp[p + 1]))
        d[idx[seg]] = val[seg]
        assert not np.any(val[seg] == marker)
        dense.append(torch.from_numpy(d.view(np.int16)).reshape(plan.tensor_shapes[p]))
    sliced = [torch.full((n,), -1, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, dense, sliced)
    for k in range(plan.n_shards):
        want = sliced[k].numpy().view(np.uint16).copy()
        want[want == marker] = canary
        assert np.array_equal(got[k], want), plan.shard_names[k]
    # and it is what extract-with-the-plan followed by apply produces
    lists = oracle.extract(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), th, mm, vv, c)
    ref = [np.full(n, canary, np.uint16) for n in plan.shard_numels]
    oracle.apply(plan.shard_numels, *lists, ref)
    for k in range(plan.n_shards):
        assert np.array_equal(got[k], ref[k])


def test_canonical_mapping_skips_other_receivers_and_reports_bad_entries():
    plan = plans.qwen3_dense_plan(1, 2, False, configs.SMALL_DENSE)
    th, mm, vv, c = _all_changed_state(plan)
    lp, idx, val = _canonical_lists(plan, th, mm, vv, c)
    mine = [k for k, r in enumerate(plan.shard_receivers) if r == 1]
    shards = [np.zeros(n, np.uint16) if k in mine else None for k, n in enumerate(plan.shard_numels)]
    oracle.apply_canonical(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), lp, idx, val, shards)
    full = [torch.zeros(n, dtype=torch.int16) for n in plan.shard_numels]
    plans.scatter_dense(plan, [_bf16_bits_t(t) for t in th], full)
    for k in mine:
        assert np.array_equal(shards[k], full[k].numpy().view(np.uint16))
    bad = idx.copy()
    bad[0] = plan.numel(0)                                   # one past the end of tensor 0
    with pytest.raises(ValueError):
        oracle.apply_canonical(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), lp, bad, val, shards)


def test_nonfinite_slots_are_counted_once_per_receiver_copy():
    """The count of receiver slots whose reconstruction is NaN, or Inf from a finite theta_t, against an
    element-wise numpy fp32 evaluation of Eq. 2 (separately rounded operations) and the plan's
    replication: a sharded tensor counts once, a replicated one once per receiver."""
    rng = np.random.default_rng(5)
    n = 4096
    th = (rng.standard_normal(n) * 0.02).astype(np.float32)
    mm = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    vv = np.abs(rng.standard_normal(n) * 1e-6).astype(np.float32)
    th[[3, 700]] = np.nan
    th[[9, 1500]] = [np.inf, -np.inf]
    vv[[20, 21, 3000]] = -1e-6                      # sqrt of a negative: NaN reconstruction
    mm[[40, 41]] = [3e38, -3e38]                    # the update overflows: Inf reconstruction
    vv[[40, 41]] = 1e-30
    c = oracle.derive_constants(7, 1e-2, 0.9, 0.999, 1e-8, 0.1)
    with np.errstate(all="ignore"):
        mhat = mm / c[0]
        den = np.sqrt(vv / c[1]) + c[4]
        prev = (th + c[3] * (mhat / den)) / c[2]
    odd = np.isnan(prev) | (np.isinf(prev) & np.isfinite(th))
    assert odd.sum() == 7 and np.isinf(prev[[9, 1500]]).all()      # the two infinite weights stay infinite: not counted
    # tensor 0: rows split over two receivers; tensor 1 (same data): replicated on three
    shapes = [(64, 64), (64, 64)]
    numels = [2048, 2048, 4096, 4096, 4096]
    ops = [(0, 0, 0, 0, 32, 64, 0, 64, 0, 0), (0, 1, 32, 0, 32, 64, 0, 64, 0, 0)] + \
          [(1, 2 + r, 0, 0, 64, 64, 0, 64, 0, 0) for r in range(3)]
    res = oracle.extract(shapes, numels, ops, [th, th], [mm, mm], [vv, vv], c, with_nonfinite=True)
    assert res[3] == int(odd.sum()) * (1 + 3)
    # and nothing is counted when everything is finite
    ok = np.where(odd, np.float32(0.01), th)
    res = oracle.extract(shapes, numels, ops, [ok, ok], [np.zeros_like(mm)] * 2, [np.abs(vv)] * 2, c, with_nonfinite=True)
    assert res[3] == 0
