"""The storage-mediated path end to end on the GPU (Section 4.4), against the oracle: extract over
the identity plan (canonical pairs), serialise, read back and verify, then map the entries into a
receiver's inference layout and store them - the result must be what the same-cluster path
(extract with the receiver plan + apply) leaves in the shards, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from gpu_util import assert_lists_equal, oracle_extract, run_extract
from synth import configs, plans
from synth.tensors import Hyper, Spec

pytestmark = pytest.mark.gpu

def _many_small_tensors(n_tensors=4200):
    """More tensors and more lists than the apply kernels keep list boundaries for in shared memory
    (4096): boundaries then come from global memory."""
    p = plans.Plan()
    for i in range(n_tensors):
        t = p.add_tensor(f"w{i}", (4, 96))
        for r in range(2):
            k = p.add_shard(f"w{i}.{r}", r, 2 * 96)
            p.add_op(t, k, (2 * r, 0), (2, 96), 0, 96, (0, 0))
    return p


PLANS = {
    "many_small_tensors": _many_small_tensors,
    "dense_tp4": lambda: plans.qwen3_dense_plan(2, 4, True, configs.SMALL_DENSE),
    "moe_tp8_ep4": lambda: plans.qwen3_moe_plan(1, 8, 4, configs.SMALL_MOE),
    "random3": lambda: plans.random_plan(1003),
    "random17": lambda: plans.random_plan(1017),
    "random22": lambda: plans.random_plan(1022),
}


def _host(lst):
    return [t.cpu().numpy() for t in lst]


@pytest.mark.parametrize("name", list(PLANS))
def test_canonical_entries_mapped_on_the_destination(name):
    plan = PLANS[name]()
    hp = Hyper(step=120, lr=2e-5, wd=0.05)
    wl = configs.Workload(name, plan, hp, [Spec()] * plan.n_tensors if name.startswith("random") else configs._specs(plan), 31)
    st = wl.materialize("cuda")
    ident = plans.canonical_plan(plan.tensor_names, plan.tensor_shapes)
    lay_c, d_c = run_extract(ident, st, hp)                       # sender: canonical (index, value) pairs
    # the oracle works on its own canonical lists (which the GPU's must equal), never on GPU output
    lp, idx, val = oracle_extract(ident, st, hp)
    assert_lists_equal(d_c.to_host(), (lp, idx, val), ident)
    assert int(lp[-1]) > 0

    lay = dte.Layout.from_plan(plan, 0)                           # destination: its plan, its shards
    canary = 0x5A5A
    shards = [torch.full((n,), canary, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply_canonical(lay, d_c, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert d_c.status_bits() == 0
    want = [np.full(n, canary, np.uint16) for n in plan.shard_numels]
    oracle.apply_canonical(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), lp, idx, val, want)
    for k in range(plan.n_shards):
        assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), want[k]), plan.shard_names[k]

    # the same-cluster path on the same state leaves the same shards
    lay2, d2 = run_extract(plan, st, hp, layout=lay)
    direct = [torch.full((n,), canary, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply(lay, d2, lay.shard_table(direct))
    torch.cuda.synchronize()
    for k in range(plan.n_shards):
        assert torch.equal(direct[k], shards[k]), plan.shard_names[k]


def test_one_receiver_passes_only_its_own_shards():
    plan = plans.qwen3_dense_plan(1, 4, True, configs.SMALL_DENSE)
    hp = Hyper(step=120, lr=2e-5, wd=0.05)
    wl = configs.Workload("recv", plan, hp, configs._specs(plan), 32)
    st = wl.materialize("cuda")
    ident = plans.canonical_plan(plan.tensor_names, plan.tensor_shapes)
    _, d_c = run_extract(ident, st, hp)
    lp, idx, val = oracle_extract(ident, st, hp)
    assert_lists_equal(d_c.to_host(), (lp, idx, val), ident)
    lay = dte.Layout.from_plan(plan, 0)
    for r in (0, 3):
        mine = [k for k, rr in enumerate(plan.shard_receivers) if rr == r]
        shards = [torch.zeros(n, dtype=torch.int16, device="cuda") if k in mine else None
                  for k, n in enumerate(plan.shard_numels)]
        dte.dte_apply_canonical(lay, d_c, lay.shard_table(shards))
        torch.cuda.synchronize()
        assert d_c.status_bits() == 0
        want = [np.zeros(n, np.uint16) if k in mine else None for k, n in enumerate(plan.shard_numels)]
        oracle.apply_canonical(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), lp, idx, val, want)
        for k in mine:
            assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), want[k])


def test_bad_canonical_entries_are_flagged_not_written():
    plan = plans.single_matrix_plan(64, 48, 2)
    lay = dte.Layout.from_plan(plan, 0)
    lp = np.array([0, 3], np.uint64)
    idx = np.array([5, 64 * 48, 100], np.uint32)              # the second index is one past the tensor
    val = np.array([1, 2, 3], np.uint16)
    d = dte.Delta.wrap(lp, torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(val.view(np.int16)).cuda())
    shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply_canonical(lay, d, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert d.status_bits() == dte.DTE_DEV_BOUNDS
    got = torch.cat(shards).cpu().numpy()
    assert got[5] == 1 and got[100] == 3 and int((got != 0).sum()) == 2
    # a delta read from a damaged stream is refused as a whole
    d.counters[2] = dte.DTE_DEV_CORRUPT
    shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply_canonical(lay, d, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert not bool(torch.cat(shards).any())


def test_entries_for_a_missing_shard_are_flagged_by_apply():
    plan = plans.single_matrix_plan(64, 48, 2)
    wl = configs.Workload("null", plan, Hyper(step=10, lr=1e-4, wd=0.0), [Spec()], 33)
    st = wl.materialize("cuda")
    lay, d = run_extract(plan, st, wl.hp)
    assert all(int(x) > 0 for x in np.diff(d.to_host()[0]))
    shards = [torch.zeros(plan.shard_numels[0], dtype=torch.int16, device="cuda"), None]
    dte.dte_apply(lay, d, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert d.status_bits() == dte.DTE_DEV_BOUNDS and bool(shards[0].any())


@pytest.mark.parametrize("fmt", [dte.DTE_CHUNK_PLAIN, dte.DTE_CHUNK_BYTE_PLANES, dte.DTE_CHUNK_DELTA_PLANES])
def test_whole_storage_path_extract_pack_unpack_map_store(fmt):
    plan = plans.qwen3_moe_plan(1, 4, 4, configs.SMALL_MOE)
    hp = Hyper(step=300, lr=1e-5, wd=0.01)
    wl = configs.Workload("storage", plan, hp, configs._specs(plan), 34)
    st = wl.materialize("cuda")
    ident = plans.canonical_plan(plan.tensor_names, plan.tensor_shapes)
    lay_c, d_c = run_extract(ident, st, hp)
    cs = dte.ChunkStream(lay_c.num_lists, d_c.total(), 512, fmt, lay_c.device)
    dte.dte_pack_chunks(lay_c, d_c, cs)
    stream, directory, info = cs.to_host()                     # what would be published
    # ---- destination: only the bytes, the directory and the list boundaries cross over ----------
    lp = d_c.list_ptr.cpu()
    dev_stream = torch.from_numpy(np.concatenate([stream, np.zeros((-stream.size) % 16 + 16, np.uint8)])).cuda()
    dev_dir = torch.from_numpy(directory.view(np.int64).copy()).cuda()
    lay_dst_c = dte.Layout.from_plan(ident, 0)
    recv = lay_dst_c.new_delta(int(lp[-1]))
    recv.list_ptr.copy_(lp)
    dte.dte_unpack_chunks(lay_dst_c, dev_stream, dev_dir, int(info[0]), recv, nbytes=stream.size)
    lay = dte.Layout.from_plan(plan, 0)
    shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply_canonical(lay, recv, lay.shard_table(shards))
    torch.cuda.synchronize()
    assert recv.counters.cpu().tolist() == [int(lp[-1]), int(info[0]), 0, 0]
    # oracle: the same chain on the host
    c = oracle.derive_constants(*hp.as_args())
    o_lp, o_idx, o_val = oracle.extract(ident.tensor_shapes, ident.shard_numels, ident.ops_array(),
                                        _host(st.theta), _host(st.m), _host(st.v), c)
    o_stream, o_dir = oracle.pack_chunks(o_lp, o_idx, o_val, 512, fmt)
    assert np.array_equal(stream, o_stream)
    u_idx, u_val, rejected, _ = oracle.unpack_chunks(o_stream, o_dir, o_lp)
    assert rejected == 0
    want = [np.zeros(n, np.uint16) for n in plan.shard_numels]
    oracle.apply_canonical(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), o_lp, u_idx, u_val, want)
    for k in range(plan.n_shards):
        assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), want[k]), plan.shard_names[k]
