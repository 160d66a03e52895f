"""GPU parity of the chunk codec (storage-mediated path, Section 4.4) against the oracle:
the serialised bytes and the directory are compared byte for byte, the reader entry by entry,
on extract results and on seeded synthetic lists that span several full chunks, ragged tails
and empty lists; damaged streams must be rejected exactly where the oracle rejects them."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from gpu_util import assert_lists_equal, oracle_extract, run_extract
from synth import configs, plans
from synth.tensors import Hyper

pytestmark = pytest.mark.gpu


def _layout(n_lists, numel=1 << 26):
    plan = plans.canonical_plan([f"t{i}" for i in range(n_lists)], [(numel, 1)] * n_lists)
    return dte.Layout.from_plan(plan, 0)


def _delta_from_lists(lay, lp, off, val, capacity=None):
    d = lay.new_delta(int(lp[-1]) if capacity is None else capacity)
    n = int(lp[-1])
    d.list_ptr.copy_(torch.from_numpy(lp.astype(np.int64)))
    if n:
        d.offsets[:n].copy_(torch.from_numpy(off.view(np.int32)))
        d.values[:n].copy_(torch.from_numpy(val.view(np.int16)))
    d.counters.zero_()
    d.counters[0] = n
    return d


def _synthetic_lists(seed, lens, numel=1 << 26):
    rng = np.random.default_rng(seed)
    lp = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    parts = [np.sort(rng.choice(numel, int(n), replace=False)).astype(np.uint32) for n in lens]
    off = np.concatenate(parts + [np.zeros(0, np.uint32)])
    val = rng.integers(0, 1 << 16, off.size).astype(np.uint16)
    return lp, off, val


def _dir_rows(directory):
    return np.stack([directory["byte_offset"], directory["list"].astype(np.uint64),
                     directory["first_entry"].astype(np.uint64)], axis=1)


def _pack(lay, d, chunk_entries, fmt, entries=None):
    cs = dte.ChunkStream(lay.num_lists, d.capacity if entries is None else entries, chunk_entries, fmt, lay.device)
    dte.dte_pack_chunks(lay, d, cs)
    torch.cuda.synchronize()
    return cs


def _unpack(lay, stream, rows, lp, prefill=0):
    n_chunks = rows.shape[0] - 1
    rec = np.zeros(n_chunks + 1, dte.CHUNK_REF_DTYPE)
    rec["byte_offset"], rec["list"], rec["first_entry"] = rows[:, 0], rows[:, 1], rows[:, 2]
    pad = (-stream.size) % 16
    dev_stream = torch.from_numpy(np.concatenate([stream, np.zeros(pad + 16, np.uint8)])).cuda()
    dev_dir = torch.from_numpy(rec.view(np.int64).copy()).cuda()
    d = lay.new_delta(max(1, int(lp[-1])))
    d.offsets.fill_(prefill)
    d.values.fill_(prefill)
    d.list_ptr.copy_(torch.from_numpy(lp.astype(np.int64)))
    dte.dte_unpack_chunks(lay, dev_stream, dev_dir, n_chunks, d, nbytes=stream.size)
    torch.cuda.synchronize()
    n = int(lp[-1])
    return (d.offsets[:n].cpu().numpy().view(np.uint32), d.values[:n].cpu().numpy().view(np.uint16),
            d.counters.cpu().numpy().astype(np.uint64), d)


@pytest.mark.parametrize("fmt", [dte.DTE_CHUNK_PLAIN, dte.DTE_CHUNK_BYTE_PLANES, dte.DTE_CHUNK_DELTA_PLANES])
@pytest.mark.parametrize("chunk_entries", [8, 64, 4096])
def test_pack_of_an_extract_result_is_byte_identical(fmt, chunk_entries):
    dense = plans.qwen3_dense_plan(1, 1, True, configs.SMALL_DENSE)
    plan = plans.canonical_plan(dense.tensor_names, dense.tensor_shapes)
    wl = configs.Workload("canonical", plan, Hyper(step=200, lr=2e-6, wd=0.05), configs._specs(plan), 77)
    st = wl.materialize("cuda")
    lay, d = run_extract(plan, st, wl.hp)
    # the oracle's writer is fed the oracle's own lists (which the GPU's must equal), never GPU output
    lp, off, val = oracle_extract(plan, st, wl.hp)
    assert_lists_equal(d.to_host(), (lp, off, val), plan)
    assert int(lp[-1]) > 1000
    cs = _pack(lay, d, chunk_entries, fmt)
    stream, directory, info = cs.to_host()
    want_stream, want_dir = oracle.pack_chunks(lp, off, val, chunk_entries, fmt)
    assert info.tolist() == [want_dir.shape[0] - 1, want_stream.size, 0, int(lp[-1])]
    assert np.array_equal(_dir_rows(directory), want_dir)
    assert np.array_equal(stream, want_stream)
    # and back, through the GPU reader, into a shard: Eq. 7 on the destination
    o2, v2, counters, d2 = _unpack(lay, stream, want_dir, lp)
    assert counters.tolist() == [int(lp[-1]), want_dir.shape[0] - 1, 0, 0]
    assert np.array_equal(o2, off) and np.array_equal(v2, val)
    shards = [torch.zeros(n, dtype=torch.int16, device="cuda") for n in plan.shard_numels]
    dte.dte_apply(lay, d2, lay.shard_table(shards))
    torch.cuda.synchronize()
    want = [np.zeros(n, np.uint16) for n in plan.shard_numels]
    oracle.apply(plan.shard_numels, lp, off, val, want)
    for k in range(len(shards)):
        assert np.array_equal(shards[k].cpu().numpy().view(np.uint16), want[k])


@pytest.mark.parametrize("fmt", [0, 1, 2])
def test_full_chunks_ragged_tails_and_empty_lists(fmt):
    lens = [200_003, 0, 65_536, 1, 0, 131_079, 7]
    lp, off, val = _synthetic_lists(11, lens)
    lay = _layout(len(lens))
    d = _delta_from_lists(lay, lp, off, val)
    cs = _pack(lay, d, 65536, fmt)
    stream, directory, info = cs.to_host()
    want_stream, want_dir = oracle.pack_chunks(lp, off, val, 65536, fmt)
    assert want_dir.shape[0] - 1 == 4 + 1 + 1 + 3 + 1
    assert info.tolist() == [want_dir.shape[0] - 1, want_stream.size, 0, int(lp[-1])]
    assert np.array_equal(_dir_rows(directory), want_dir)
    assert np.array_equal(stream, want_stream)
    o2, v2, counters, _ = _unpack(lay, want_stream, want_dir, lp)
    assert counters.tolist() == [int(lp[-1]), want_dir.shape[0] - 1, 0, 0]
    assert np.array_equal(o2, off) and np.array_equal(v2, val)


def test_many_lists_cross_the_planner_block():
    # more lists than the planning CTA has threads, most of them empty or tiny
    rng = np.random.default_rng(4)
    lens = rng.integers(0, 40, 2500)
    lens[rng.random(2500) < 0.4] = 0
    lp, off, val = _synthetic_lists(12, lens, numel=1 << 16)
    lay = _layout(len(lens), numel=1 << 16)
    d = _delta_from_lists(lay, lp, off, val)
    for fmt in (0, 1, 2):
        stream, directory, info = _pack(lay, d, 16, fmt).to_host()
        want_stream, want_dir = oracle.pack_chunks(lp, off, val, 16, fmt)
        assert np.array_equal(_dir_rows(directory), want_dir)
        assert np.array_equal(stream, want_stream)


def test_empty_delta_and_overflow_reports():
    lay = _layout(3)
    lp = np.zeros(4, np.uint64)
    d = _delta_from_lists(lay, lp, np.zeros(0, np.uint32), np.zeros(0, np.uint16), capacity=8)
    stream, directory, info = _pack(lay, d, 64, 0).to_host()
    assert info.tolist() == [0, 0, 0, 0] and stream.size == 0
    assert _dir_rows(directory).tolist() == [[0, 0xFFFFFFFF, 0]]
    # directory / stream too small: nothing written, exact requirement reported
    lp, off, val = _synthetic_lists(13, [1000, 0, 300])
    d = _delta_from_lists(lay, lp, off, val)
    want_stream, want_dir = oracle.pack_chunks(lp, off, val, 64, 1)
    cs = dte.ChunkStream(lay.num_lists, 64, 64, 1, lay.device)      # sized for 64 entries only
    cs.stream.fill_(0xAB)
    dte.dte_pack_chunks(lay, d, cs)
    torch.cuda.synchronize()
    info = cs.info.cpu().numpy()
    assert info[:3].tolist() == [want_dir.shape[0] - 1, want_stream.size, dte.DTE_DEV_OVERFLOW]
    assert bool((cs.stream == 0xAB).all())
    # an overflowed delta is not serialised
    d.counters[2] = dte.DTE_DEV_OVERFLOW
    cs = _pack(lay, d, 64, 1)
    assert cs.info.cpu().numpy().tolist() == [0, 0, dte.DTE_DEV_OVERFLOW, 0]


def test_bad_arguments_are_rejected_on_the_host():
    lay = _layout(2)
    d = lay.new_delta(16)
    for chunk_entries, fmt in ((12, 0), (0, 0), (1 << 21, 0), (64, 3)):
        cs = dte.ChunkStream(2, 16, 64, 0, lay.device)
        cs.chunk_entries, cs.format = chunk_entries, fmt
        with pytest.raises(dte.DteError) as e:
            dte.dte_pack_chunks(lay, d, cs)
        assert e.value.status == 1


@pytest.mark.parametrize("fmt", [0, 1, 2])
def test_damaged_streams_are_rejected_where_the_oracle_rejects_them(fmt):
    lens = [150, 0, 70, 33]
    numel = 1 << 20
    lp, off, val = _synthetic_lists(14, lens, numel)
    lay = _layout(len(lens), numel)
    shard = torch.full((numel,), 7, dtype=torch.int16, device="cuda")   # every list's destination
    stream, rows = oracle.pack_chunks(lp, off, val, 64, fmt)
    n_chunks = rows.shape[0] - 1
    rng = np.random.default_rng(15)
    cases = []
    for _ in range(24):                                   # one flipped bit anywhere in the stream
        bad = stream.copy()
        pos = int(rng.integers(0, stream.size))
        bad[pos] ^= np.uint8(1 << int(rng.integers(0, 8)))
        cases.append((bad, rows))
    for c in range(n_chunks):                             # every checked header byte of every chunk
        for b in range(0, 28, 3):
            bad = stream.copy()
            bad[int(rows[c, 0]) + b] ^= 0x10
            cases.append((bad, rows))
    for row, col, value in ((1, 0, int(rows[1, 0]) + 8), (n_chunks, 0, stream.size + 32), (2, 0, int(rows[1, 0]) + 16),
                            (0, 1, 2), (1, 2, 8), (3, 1, 9)):   # the directory misplaces or mislabels a chunk
        bad_rows = rows.copy()
        bad_rows[row, col] = value
        cases.append((stream, bad_rows))
    seen_rejections = 0
    for bad, bad_rows in cases:
        want_off, want_val, want_rej, want_written = oracle.unpack_chunks(bad, bad_rows, lp)
        o2, v2, counters, d2 = _unpack(lay, bad, bad_rows, lp)
        assert counters[3] == want_rej and counters[0] == want_written and counters[1] == n_chunks - want_rej
        assert bool(counters[2] & dte.DTE_DEV_CORRUPT) == (want_rej > 0)
        assert np.array_equal(o2, want_off) and np.array_equal(v2, want_val)
        seen_rejections += want_rej
        if want_rej:                                      # apply must not touch the shards
            dte.dte_apply(lay, d2, lay.shard_table([shard] * len(lens)))
            torch.cuda.synchronize()
            assert bool((shard == 7).all())
    assert seen_rejections >= len(cases) - 8              # reserved header bytes may be flipped unnoticed


def test_list_boundaries_that_do_not_nest_are_rejected():
    lens = [100, 50]
    lp, off, val = _synthetic_lists(21, lens, 1 << 20)
    lay = _layout(2, 1 << 20)
    stream, rows = oracle.pack_chunks(lp, off, val, 64, 1)
    bad_lp = lp.copy()
    bad_lp[1] = 1 << 40                                   # list 0 "ends" far outside the buffers
    o2, v2, counters, _ = _unpack(lay, stream, rows, bad_lp)
    assert counters[0] == 0 and counters[3] == rows.shape[0] - 1 and counters[2] & dte.DTE_DEV_CORRUPT
