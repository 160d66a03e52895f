"""Every fp32 bit pattern of theta, once: a 65536 x 65536 source tensor whose element i has the
bit pattern i, with moments that cycle through small tables (signs, magnitudes from far below to
far above the distance to a BF16 rounding boundary, zeros, a negative and a subnormal second
moment).  The changed set, offsets and values of the CUDA path must equal the oracle's Eq. 4 mask
on all 2^32 elements - NaNs, infinities, subnormals, ties and the overflow threshold included -
for hyper-parameters with and without the divisions by the bias correction and the decay factor.
The same for every bit pattern of the first moment and of the second moment, theta then cycling
through weights, ties, zeros and extremes.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import paper_2608_00455_b200 as dte
from synth import plans

pytestmark = pytest.mark.gpu

N = 1 << 32
HALF = 1 << 31
CHUNK = 1 << 25
M_TABLE = np.array([3e-4, -3e-4, 1e-6, -2e-2, 0.0, 5e-9, -1.5e-3], np.float32)            # period 7
V_TABLE = np.array([1e-6, 4e-10, 0.0, 2.5e-3, 1e-40, -1e-6, 9e-8, 1e-12, 3e-5, 1e-6, 6e-7], np.float32)   # period 11


# theta when it is not the exhaustive operand: weights, BF16 ties and their neighbours, zeros,
# the overflow threshold, a subnormal tie, +-65504                                             period 13
T_TABLE = np.array([0x3C23D70A, 0xBCA3D70A, 0x3F808000, 0x3F807FFF, 0x3F808001, 0x00000000, 0x80000000,
                    0x7F7F8000, 0x00008000, 0x3F800000, 0xC77FE000, 0x3A83126F, 0xBF818000], np.uint32).view(np.float32)


# A second pair of moment tables for the run with a decay far from 1 (0.9): there the division
# moves every normal theta out of its BF16 cell, and the decision is at its threshold only in the
# lowest BF16 cells (|theta| < 2^-126), where a cell is as wide as its values.  These moments give
# steps of 0 and of about a quarter, one and three of those cells (2^-133) next to ordinary ones.
M_TABLE_TINY = np.array([1.4e-30, -1.4e-30, 0.0, 5.6e-30, -1.7e-29, 3e-4, -3e-31], np.float32)          # period 7
V_TABLE_TINY = np.array([1e18, 1e18, 1e-6, 1e18, 4e18, 1e18, 0.0, 1e18, 2.5e17, 1e18, 1e18], np.float32)  # period 11


def _operands(which, lo, n, tiny=False):
    """(theta, m, v) of elements lo .. lo+n-1: operand `which` has bit pattern i, the others cycle."""
    i = np.arange(lo, lo + n, dtype=np.int64)
    exhaustive = i.astype(np.uint32).view(np.float32)
    th = exhaustive if which == "theta" else T_TABLE[i % 13]
    mm = exhaustive if which == "m" else (M_TABLE_TINY if tiny else M_TABLE)[i % 7]
    vv = exhaustive if which == "v" else (V_TABLE_TINY if tiny else V_TABLE)[i % 11]
    return th, mm, vv


HP_PLAIN = (500, 1e-6, 0.9, 0.999, 1e-8, 0.01)     # bc1 = decay = 1: no constant division
HP_DECAY = (3, 2e-4, 0.9, 0.999, 1e-8, 0.1)         # both divisions, direction-aware screen with decay
HP_EPS0 = (40, 1e-3, 0.8, 0.99, 0.0, 0.0)           # eps = 0: m = v = 0 gives 0/0
HP_DECAY09 = (20, 0.1, 0.9, 0.999, 1e-8, 1.0)       # decay = 0.9, with the tiny-step tables


@pytest.mark.parametrize("which,hp", [("theta", HP_PLAIN), ("theta", HP_DECAY), ("theta", HP_EPS0),
                                      ("m", HP_DECAY), ("v", HP_DECAY), ("v", HP_PLAIN), ("theta", HP_DECAY09)],
                         ids=["theta-plain", "theta-decay", "theta-eps0", "m-decay", "v-decay", "v-plain",
                              "theta-decay0.9-tiny-steps"])
def test_every_fp32_pattern_of_one_operand(which, hp):
    free, _ = torch.cuda.mem_get_info()
    if free < 110e9:
        pytest.skip("needs 110 GB of free device memory")
    dev = torch.device("cuda", 0)
    theta = torch.empty(N, dtype=torch.float32, device=dev)
    m = torch.empty(N, dtype=torch.float32, device=dev)
    v = torch.empty(N, dtype=torch.float32, device=dev)
    tiny = hp is HP_DECAY09
    tt, mt, vt = (torch.from_numpy(x.copy()).to(dev)
                  for x in (T_TABLE, M_TABLE_TINY if tiny else M_TABLE, V_TABLE_TINY if tiny else V_TABLE))
    for lo in range(0, N, 1 << 28):
        sl = slice(lo, lo + (1 << 28))
        i = torch.arange(lo, lo + (1 << 28), dtype=torch.int64, device=dev)
        bits = (i if lo < HALF else i - N).to(torch.int32).view(torch.float32)      # element i has bit pattern i
        theta[sl] = bits if which == "theta" else tt[i % 13]
        m[sl] = bits if which == "m" else mt[i % 7]
        v[sl] = bits if which == "v" else vt[i % 11]
        del i, bits
    probe = {"theta": theta, "m": m, "v": v}[which]
    assert int(probe[12345].view(torch.int32)) == 12345 and int(probe[N - 1].view(torch.int32)) == -1
    # two receivers, 2^31 elements each (a destination tensor must have fewer than 2^32)
    plan = plans.Plan()
    a = plan.add_tensor("all", (1 << 16, 1 << 16))
    for r in range(2):
        k = plan.add_shard(f"half{r}", r, HALF)
        plan.add_op(a, k, (r << 15, 0), (1 << 15, 1 << 16), 0, 1 << 16, (0, 0))
    lay = dte.Layout.from_plan(plan, 0)
    assert lay.num_elements == N
    # size discovery first (with theta exhaustive about half of all patterns change: every theta
    # smaller than the step does), then buffers of exactly that size
    tabs = lay.source_tables([theta], [m], [v])
    d = lay.new_delta(1024)
    dte.dte_extract_delta(lay, tabs, *hp, d)
    torch.cuda.synchronize()
    assert d.status_bits() == dte.DTE_DEV_OVERFLOW
    total = d.total()
    assert N // 1000 < total < N
    d = lay.new_delta(total)
    dte.dte_extract_delta(lay, tabs, *hp, d)
    torch.cuda.synchronize()
    assert d.status_bits() == 0 and d.total() == total
    del theta, m, v
    torch.cuda.empty_cache()
    lp = d.list_ptr.cpu().numpy().astype(np.int64)
    consts = oracle.derive_constants(*hp)

    def job(lo):
        th, mm, vv = _operands(which, lo, CHUNK, tiny)
        mask, v16 = oracle.changed_mask(th, mm, vv, consts)
        idx = np.nonzero(mask)[0]
        prev = oracle.invert(th, mm, vv, consts)
        odd = int((np.isnan(prev) | (np.isinf(prev) & np.isfinite(th))).sum())
        return lo, (idx + (lo % HALF)).astype(np.uint32), v16[idx], odd

    cursor, odd_total = 0, 0
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as pool:
        for lo, want_off, want_val, odd in pool.map(job, range(0, N, CHUNK)):
            odd_total += odd
            if lo == HALF:
                assert cursor == int(lp[1]), "boundary between the two lists"
            n = want_off.size
            assert cursor + n <= total, f"more entries expected than produced, chunk at {lo:#x}"
            off = d.offsets[cursor:cursor + n].cpu().numpy().view(np.uint32)
            val = d.values[cursor:cursor + n].cpu().numpy().view(np.uint16)
            assert np.array_equal(off, want_off), f"offsets of chunk at {lo:#x}"
            assert np.array_equal(val, want_val), f"values of chunk at {lo:#x}"
            cursor += n
    assert cursor == total
    # reconstructions that are NaN (NaN operands, negative v, 0/0) or overflowed were all counted
    assert int(d.counters[3].item()) == odd_total and odd_total >= (1 << 24)
