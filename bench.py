#!/usr/bin/env python
"""Benchmark of the delta-transfer hot path on synthetic Qwen3-8B-shaped optimizer state.

One step = one pass of the whole path over the resident state: the fused extract kernel
(AdamW inversion, BF16 compare, ordered compaction, receiver remap) followed by the apply
kernel on the receiver shard buffers.  Prints one JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload full|layers:L|config1|config4]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

With N > 1 (torchrun) every rank runs the same per-GPU workload on its own device: the
path partitions by tensor with no data-path collective, so this is weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from synth import configs, plans  # noqa: E402

METRIC = "delta_extract_scanned_GBps"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
# Measured DRAM traffic of the extract kernel (ncu: dram__bytes_read.sum + dram__bytes_write.sum
# of one launch over a one-layer case, and the elements that launch scanned), kept as data next
# to the capture's summary; `roofline.traffic` scales it to the workload's element count.
EXTRACT_TRAFFIC_JSON = os.path.join(ROOT, "profiles", "extract_kernel.qwen3-8b-one-layer.traffic.json")
APPLY_TRAFFIC_JSON = os.path.join(ROOT, "profiles", "apply_kernel.qwen3-8b-one-layer.traffic.json")


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        rows = [r for t, r in self.rows if t0 <= t <= t1] or [r for _, r in self.rows[-3:]]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except Exception:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def build_workload(name: str, device):
    if name == "full":
        return configs.config3(device)
    if name.startswith("layers:"):
        return configs.config3(device, n_layers=int(name.split(":")[1]), with_embeddings=False)
    if name.startswith("mcore:"):        # mcore:<sender TP>:<receiver TP>:<dp slices>[:<layers>]
        f = [int(x) for x in name.split(":")[1:]]
        return configs.config3_mcore(device, f[0], f[1], f[2], n_layers=f[3] if len(f) > 3 else 36)
    if name == "config1":
        return configs.config1()
    if name == "config2":
        return configs.config2()
    if name == "config4":
        return configs.config4(device)
    if name.startswith("moe:"):          # moe:<receiver TP>:<EP>[:<layers>]  (config 4's state, other inference layout)
        f = [int(x) for x in name.split(":")[1:]]
        return configs.config4(device, n_layers=f[2] if len(f) > 2 else 12, tp=f[0], ep=f[1])
    if name.startswith("sweep:"):        # sweep:<lr>:<sigma_g>  (one point of the density sweep, t=100, wd=0.01)
        f = name.split(":")[1:]
        return configs.config5(float(f[0]), 100, 0.01, float(f[1]))
    raise SystemExit(f"unknown workload {name}")


def materialize_resident(wl, device, dte):
    """theta/m/v resident on the device; shards initialised to remapped BF16(true theta_{t-1})."""
    plan = wl.plan
    shards = [torch.zeros(n, dtype=torch.int16, device=device) for n in plan.shard_numels]
    ops_by_tensor = {}
    for o in plan.ops:
        ops_by_tensor.setdefault(o[0], []).append(o)
    st = configs.State([None] * plan.n_tensors, [None] * plan.n_tensors, [None] * plan.n_tensors,
                       [None] * plan.n_tensors)
    alias = wl.alias_of or list(range(plan.n_tensors))
    members = {}
    for p, a in enumerate(alias):
        members.setdefault(a, []).append(p)
    for base, group in members.items():
        one = wl.materialize(device, [base])
        prev = one.prev_bf16[base].view(torch.int16).reshape(plan.tensor_shapes[base])
        for p in group:                  # slices of one shard share its allocation
            st.theta[p], st.m[p], st.v[p] = one.theta[base], one.m[base], one.v[base]
            for (_, dst, a0, a1, e0, e1, b0, ld, r0, r1) in ops_by_tensor.get(p, []):
                shards[dst].as_strided((e0, e1), (ld, 1), b0 + r0 * ld + r1).copy_(prev[a0:a0 + e0, a1:a1 + e1])
        del one, prev
    return st, shards


def reconstruction_vs_truth(plan, st, shards_after, init_vals, delta_host):
    """FN = truly changed but not emitted (receiver left stale); FP = emitted but not truly changed."""
    lp, off, val = delta_host
    fp = 0
    for k in range(plan.n_shards):
        a, b = int(lp[k]), int(lp[k + 1])
        if b > a:
            fp += int((init_vals[a:b] == val[a:b]).sum().item())
    ops_by_shard = {}
    for o in plan.ops:
        ops_by_shard.setdefault(o[1], []).append(o)
    fn = 0
    for k in range(plan.n_shards):
        exp = torch.zeros_like(shards_after[k])
        for (src, _, a0, a1, e0, e1, base, ld, r0, r1) in ops_by_shard.get(k, []):
            s2 = st.theta[src].reshape(plan.tensor_shapes[src])[a0:a0 + e0, a1:a1 + e1]
            exp.as_strided((e0, e1), (ld, 1), base + r0 * ld + r1).copy_(s2.to(torch.bfloat16).view(torch.int16))
        fn += int((exp != shards_after[k]).sum().item())
        del exp
    return fn, fp


def oracle_sample(wl, st, max_elements):
    """Source tensors (in order) up to max_elements, copied to the host for the oracle."""
    plan = wl.plan
    chosen, n = [], 0
    for p in range(plan.n_tensors):
        if n + plan.numel(p) > max_elements and chosen:
            break
        chosen.append(p)
        n += plan.numel(p)
    return chosen, n


def oracle_inputs(plan, st, chosen):
    """Host arrays and the sub-plan (operations of the chosen tensors) in the oracle's format."""
    ops = plan.ops_array()
    ops = ops[np.isin(ops[:, 0], np.asarray(chosen))]
    zero = np.zeros(0, np.float32)
    cs = set(chosen)
    shapes = [s if p in cs else (0, 1) for p, s in enumerate(plan.tensor_shapes)]
    host = [[l[p].cpu().numpy() if p in cs else zero for p in range(plan.n_tensors)]
            for l in (st.theta, st.m, st.v)]
    return shapes, ops, host


def time_oracle(wl, st, chosen):
    import oracle
    shapes, ops, host = oracle_inputs(wl.plan, st, chosen)
    c = oracle.derive_constants(*wl.hp.as_args())
    t0 = time.perf_counter()
    res = oracle.extract(shapes, wl.plan.shard_numels, ops, *host, c)
    return time.perf_counter() - t0, res


def time_oracle_threads(wl, st, chosen, threads):
    """The same single-threaded oracle on `threads` host threads, each with a disjoint share of the
    chosen tensors (largest first onto the least loaded thread); wall-clock of the slowest."""
    import threading
    import oracle
    plan = wl.plan
    shares = [[] for _ in range(threads)]
    load = [0] * threads
    for p in sorted(chosen, key=lambda q: -plan.numel(q)):
        i = load.index(min(load))
        shares[i].append(p)
        load[i] += plan.numel(p)
    shares = [sorted(s) for s in shares if s]
    c = oracle.derive_constants(*wl.hp.as_args())
    jobs = [oracle_inputs(plan, st, share) for share in shares]
    changed = [0] * len(jobs)

    def work(i):
        shapes, ops, host = jobs[i]
        changed[i] = int(oracle.extract(shapes, plan.shard_numels, ops, *host, c)[0][-1])

    ts = [threading.Thread(target=work, args=(i,)) for i in range(len(jobs))]
    t0 = time.perf_counter()
    for t in ts: t.start()
    for t in ts: t.join()
    dt = time.perf_counter() - t0
    scanned = int(sum(int((j[1][:, 4] * j[1][:, 5]).sum()) for j in jobs))
    return dt, scanned, sum(changed), len(jobs)


def extract_traffic(n_elements):
    """DRAM bytes one extract call moves for `n_elements` scanned elements, scaled from the
    committed ncu capture (traffic grows in proportion to the elements scanned)."""
    try:
        with open(EXTRACT_TRAFFIC_JSON) as f:
            t = json.load(f)
        per_el = (float(t["dram_bytes_read"]) + float(t["dram_bytes_write"])) / float(t["elements_scanned"])
        return per_el * n_elements, {"bytes_per_element": per_el, "capture": os.path.basename(EXTRACT_TRAFFIC_JSON),
                                     "scaled_from_elements": int(t["elements_scanned"])}
    except Exception as e:      # no capture committed: say so instead of inventing a number
        return None, {"error": f"{type(e).__name__}: {e}"}


def apply_traffic_per_entry():
    """DRAM bytes per entry of apply_kernel at the headline density, from the committed ncu capture
    (sector fill + write-back of the touched sectors + the lists); None without a capture."""
    try:
        with open(APPLY_TRAFFIC_JSON) as f:
            t = json.load(f)
        return (float(t["dram_bytes_read"]) + float(t["dram_bytes_write"])) / float(t["entries"])
    except Exception:
        return None


def time_leg(dte, make_wl, device, steps, warmup, peak, capacity_frac=0.03, with_clocks=True, copies=1):
    """One more workload through the same timed loop as the headline: resident state, `warmup`
    untimed steps, `steps` timed steps of extract + apply (CUDA events per step).  A state that
    could sit in the 126 MB L2 is generated `copies` times (seeds differ) and the steps rotate
    over the copies, each with a layout of its own, so that every step reads inputs the L2 does
    not hold: inputs larger than L2, and no dirty lines left behind by a flushing write.
    Returns the leg's numbers; frees its memory."""
    sets, N, names = [], 0, None
    for i in range(copies):
        wl = make_wl(i)
        plan = wl.plan
        st, shards = materialize_resident(wl, device, dte)
        lay = dte.Layout.from_plan(plan, device.index or 0)
        N = lay.num_elements
        delta = lay.new_delta(int(N * capacity_frac) + 1024)
        tabs = lay.source_tables(st.theta, st.m, st.v)
        hp = wl.hp.as_args()
        dte.dte_extract_delta(lay, tabs, *hp, delta)
        torch.cuda.synchronize()
        if delta.status_bits() & dte.DTE_DEV_OVERFLOW:       # dense sweep points: the sizes are exact, grow and repeat
            delta = lay.new_delta(delta.total() + 1024)
            dte.dte_extract_delta(lay, tabs, *hp, delta)
            torch.cuda.synchronize()
        if delta.status_bits():
            return {"workload": wl.name, "error": f"device status bits {delta.status_bits()}"}
        sets.append(dict(wl=wl, st=st, shards=shards, lay=lay, delta=delta, tabs=tabs, hp=hp,
                         shard_tab=lay.shard_table(shards), M=delta.total()))
    wl, lay, plan = sets[0]["wl"], sets[0]["lay"], sets[0]["wl"].plan
    resident = 12 * N * copies
    flush = torch.empty(1 << 28, dtype=torch.uint8, device=device) if resident < 1e9 else None
    stream = torch.cuda.current_stream()

    def step(i, ev=None):
        s = sets[i % copies]
        if ev: ev[0].record(stream)
        dte.dte_extract_delta(s["lay"], s["tabs"], *s["hp"], s["delta"])
        if ev: ev[1].record(stream)
        dte.dte_apply(s["lay"], s["delta"], s["shard_tab"])
        if ev: ev[2].record(stream)

    for i in range(max(warmup, 3, copies)):
        step(i)
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    sampler = ClockSampler(device.index or 0)
    if with_clocks:
        sampler.start()
        time.sleep(0.25)
    w0 = time.time()
    for i in range(steps):
        if flush is not None:
            flush.zero_()
        step(i, evs[i])
    torch.cuda.synchronize()
    w1 = time.time()
    clocks = sampler.stop(w0, w1) if with_clocks else None
    ext = [e[0].elapsed_time(e[1]) for e in evs]
    app = [e[1].elapsed_time(e[2]) for e in evs]
    ext_avg, app_avg = sum(ext) / len(ext), sum(app) / len(app)
    M = sum(s["M"] for s in sets) / copies
    gbps = (12.0 * N + 6.0 * M) / (ext_avg * 1e-3) / 1e9
    if flush is not None:
        l2 = "256 MB written between timed steps"
    elif copies > 1:
        l2 = f"{copies} copies of the state ({resident / 1e9:.2f} GB), one per step in rotation: inputs larger than L2"
    else:
        l2 = "inputs larger than L2"
    out = {"workload": wl.name, "elements_scanned": N, "changed": M, "changed_frac": M / N,
           "lists": lay.num_lists, "operations": len(plan.ops), "steps": steps,
           "hyper": {"step": wl.hp.step, "lr": wl.hp.lr, "wd": wl.hp.wd},
           "extract_ms": ext_avg, "extract_ms_min": min(ext), "extract_GBps": gbps, "frac_of_peak": gbps / peak,
           "apply_ms": app_avg, "apply_Mchanged_per_s": M / (app_avg * 1e-3) / 1e6 if M else None, "l2": l2,
           "gpu_launches": (lay.last_launch()["kernels"] + 1) * steps, "launch": lay.last_launch(), "clocks": clocks,
           **{k: v for k, v in wl.notes.items() if k in ("cold_experts", "sigma_g")}}
    del sets, flush, lay, wl, plan
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return out


def density_sweep_points():
    """(lr, step, wd, sigma_g) of the density / edge configuration that the benchmark times: the
    five learning rates at t = 100, wd = 0.01, and the two dense points at lr = 1e-4."""
    return [(lr, 100, 0.01, 1e-3) for lr in (1e-8, 1e-7, 1e-6, 1e-5, 1e-4)] + [(1e-4, 100, 0.01, 3e-3),
                                                                                (1e-4, 100, 0.01, 1e-2)]


def run_probes(device):
    """What the memory system does for the path's two access patterns, without the path: a
    read-only stream (extract) and isolated small accesses at ascending offsets, one per 67
    elements as at 1.5 % density (apply).  Prints one JSON line."""
    from paper_2608_00455_b200 import probes
    out = {"read_only_stream": read_ceiling(device)}
    n, stride, jitter = 60 << 20, 67, 60
    off = probes.make_offsets(n, stride, jitter, device)
    dst = torch.zeros(n * stride + 256, dtype=torch.int16, device=device)
    sink = torch.zeros(1, dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream()
    rates = {}
    for ctas in (6, 12):
        for mode, name in probes.SPARSE_MODES.items():
            ms = []
            for rep in range(6):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                probes.sparse_access(mode, off, dst, sink, ctas)
                e1.record(stream)
                torch.cuda.synchronize()
                if rep:
                    ms.append(e0.elapsed_time(e1))
            rates[f"{name}, {ctas} CTAs/SM"] = {"ms": sum(ms) / len(ms), "G_per_s": n / (sum(ms) / len(ms) * 1e-3) / 1e9}
    out["sparse_access"] = {"entries": n, "stride_elements": stride, "jitter": jitter, "element_bytes": 2,
                            "destination_bytes": int(dst.numel() * 2), "rates": rates}
    print(json.dumps(out), flush=True)


def read_ceiling(device, nbytes=4 << 30, reps=10):
    """Read-only streaming bandwidth: one launch over a 4 GiB buffer of its own (CUDA events)."""
    from paper_2608_00455_b200 import probes
    buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
    buf.random_(0, 256)
    out = torch.zeros(1, dtype=torch.int64, device=device)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        probes.read_bandwidth(buf, out)
    torch.cuda.synchronize()
    ms = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        probes.read_bandwidth(buf, out)
        e1.record(stream)
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    avg = sum(ms) / len(ms)
    return {"GBps": nbytes / (avg * 1e-3) / 1e9, "GBps_best": nbytes / (min(ms) * 1e-3) / 1e9, "bytes": nbytes,
            "launches": reps, "note": "4 GiB buffer, larger than L2, one launch per pass"}


def run_reference(args, rank):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    wl = build_workload(args.workload, dev)
    plan = wl.plan
    budget = int(args.ref_elements)
    chosen, n = [], 0
    for p in range(plan.n_tensors):
        if n + plan.numel(p) > budget and chosen:
            break
        chosen.append(p); n += plan.numel(p)
    st = wl.materialize(dev, chosen)
    import oracle
    shapes, ops, host = oracle_inputs(plan, st, chosen)
    scanned = int((ops[:, 4] * ops[:, 5]).sum())
    c = oracle.derive_constants(*wl.hp.as_args())
    times, M = [], 0
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        lp, off, val = oracle.extract(shapes, plan.shard_numels, ops, *host, c)
        # apply is part of the step: scatter into receiver-sized host buffers
        bufs = [np.zeros(nn if lp[k + 1] > lp[k] else 0, np.uint16) for k, nn in enumerate(plan.shard_numels)]
        numels = [b.size for b in bufs]
        oracle.apply(numels, lp, off, val, bufs)
        dt = time.perf_counter() - t0
        M = int(lp[-1])
        if i >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    value = (12.0 * scanned + 6.0 * M) / t / 1e9
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": wl.name, "sample": f"first {len(chosen)} source tensors, {scanned} elements per step"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                            "sample": f"first {len(chosen)} source tensors ({scanned} elements) of {wl.name}"},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "elements_per_s": scanned / t, "changed": M}
    print(json.dumps(out), flush=True)


def time_storage_path(dte, wl, st, shards, hp, capacity, device, peak, chunk_entries=16384, reps=5):
    """Storage-mediated path (Section 4.4), outside the timed step: extract over the identity plan
    (canonical index / value pairs), serialise into chunks (byte planes of index gaps), verify + read back, map into
    the receiver layout and store.  Each leg timed with CUDA events, L2 flushed before each call."""
    plan = wl.plan
    ident = plans.canonical_plan(plan.tensor_names, plan.tensor_shapes)
    lay_c = dte.Layout.from_plan(ident, device.index or 0)
    lay = dte.Layout.from_plan(plan, device.index or 0)
    used = sorted(set(int(o[0]) for o in plan.ops))
    theta = [st.theta[p] if p in used else None for p in range(plan.n_tensors)]
    d_c = lay_c.new_delta(capacity)
    tabs = lay_c.source_tables(st.theta, st.m, st.v)
    shard_tab = lay.shard_table(shards)
    stream = torch.cuda.current_stream()
    dte.dte_extract_delta(lay_c, tabs, *hp, d_c)
    torch.cuda.synchronize()
    if d_c.status_bits():
        return {"error": f"canonical extract status bits {d_c.status_bits()}"}
    M = d_c.total()
    fmt = dte.DTE_CHUNK_DELTA_PLANES
    cs = dte.ChunkStream(lay_c.num_lists, M, chunk_entries, fmt, device)
    back = lay_c.new_delta(M)
    back.list_ptr.copy_(d_c.list_ptr)
    dte.dte_pack_chunks(lay_c, d_c, cs)
    torch.cuda.synchronize()
    n_chunks, nbytes, bits, _ = (int(x) for x in cs.info.cpu().tolist())
    if bits:
        return {"error": f"pack status bits {bits}"}
    dte.dte_unpack_chunks(lay_c, cs.stream, cs.directory, n_chunks, back, nbytes=nbytes)
    dte.dte_apply_canonical(lay, back, shard_tab)      # also uploads the mapping tables (first use)
    torch.cuda.synchronize()
    flush = torch.empty(1 << 28, dtype=torch.uint8, device=device)
    legs = {
        "extract_canonical": lambda: dte.dte_extract_delta(lay_c, tabs, *hp, d_c),
        "pack": lambda: dte.dte_pack_chunks(lay_c, d_c, cs),
        "unpack": lambda: dte.dte_unpack_chunks(lay_c, cs.stream, cs.directory, n_chunks, back, nbytes=nbytes),
        "map_and_store": lambda: dte.dte_apply_canonical(lay, back, shard_tab),
    }
    ms = {k: [] for k in legs}
    for _ in range(reps):
        for k, fn in legs.items():
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.zero_()
            e0.record(stream); fn(); e1.record(stream)
            torch.cuda.synchronize()
            ms[k].append(e0.elapsed_time(e1))
    avg = {k: sum(v) / len(v) for k, v in ms.items()}
    same = bool(torch.equal(back.offsets[:M], d_c.offsets[:M]) and torch.equal(back.values[:M], d_c.values[:M]))
    counters = back.counters.cpu().tolist()
    moved = 6.0 * M + nbytes
    n_src = sum(plan.numel(p) for p in used)
    del theta
    return {"format": "byte planes of index gaps", "chunk_entries": chunk_entries, "chunks": n_chunks,
            "stream_bytes": nbytes, "entries": M, "canonical_elements": n_src,
            "extract_canonical_ms": avg["extract_canonical"],
            "extract_canonical_GBps": (12.0 * lay_c.num_elements + 6.0 * M) / (avg["extract_canonical"] * 1e-3) / 1e9,
            "pack_ms": avg["pack"], "unpack_ms": avg["unpack"], "map_and_store_ms": avg["map_and_store"],
            "pack_GBps": moved / (avg["pack"] * 1e-3) / 1e9, "unpack_GBps": moved / (avg["unpack"] * 1e-3) / 1e9,
            "pack_frac_of_peak": moved / (avg["pack"] * 1e-3) / 1e9 / peak,
            "unpack_frac_of_peak": moved / (avg["unpack"] * 1e-3) / 1e9 / peak,
            "map_and_store_Mentries_per_s": M / (avg["map_and_store"] * 1e-3) / 1e6,
            "round_trip_equal": same, "chunks_rejected": int(counters[3]), "status_bits": back.status_bits(),
            "gpu_launches": (5 + 2 + 1 + 1) * reps, "l2": "256 MB written before each timed call"}


def time_push(dte, lay, tabs, hp, delta, device, steps=10):
    """The same-cluster transfer fused into the extract (Section 4.3), outside the timed step: one
    extract call that also stores every receiver's lists, counts and status block into landing
    buffers.  This run has one GPU, so the landing buffers are local allocations: the number is the
    kernel-side cost of the second store of every entry and of the closing kernel, not NVLink time."""
    R = lay.num_receivers
    if R == 0:
        return None
    cap = delta.capacity
    try:
        targets = [dte.PushTarget(lay.num_lists, cap, lay.receiver_num_ops(r), device) for r in range(R)]
        stream = torch.cuda.current_stream()
        for i in range(2):
            dte.dte_extract_delta_push(lay, tabs, *hp, delta, targets, 100 + i)
        torch.cuda.synchronize()
        ms = []
        for i in range(steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            dte.dte_extract_delta_push(lay, tabs, *hp, delta, targets, 200 + i)
            e1.record(stream)
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        status = [t.status.cpu().tolist() for t in targets]
        delivered = [int(s[0]) for s in status]
        ok = all(int(s[1]) == 200 + steps - 1 and int(s[2]) == 0 for s in status) and sum(delivered) == delta.total()
        # the first receiver's slice must equal the head of the sender's own lists
        n0 = delivered[0]
        same = bool(torch.equal(targets[0].offsets[:n0], delta.offsets[:n0]) and
                    torch.equal(targets[0].values[:n0], delta.values[:n0]))
        return {"ms": sum(ms) / len(ms), "ms_min": min(ms), "receivers": R, "entries_delivered": delivered,
                "status_ok": bool(ok), "first_slice_equal": same, "launches_per_call": lay.last_launch()["kernels"],
                "note": "landing buffers on the same GPU (one GPU per run): kernel-side cost only, no NVLink"}
    except dte.DteError as e:
        return {"error": str(e)}


def aggregate_over_ranks(ms_local: float, units_local: float, dist, device):
    """Weak scaling: the job's time is the slowest rank's, its units the sum over ranks."""
    if dist is None:
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dte", choices=["dte", "reference"])
    ap.add_argument("--workload", default="full")
    ap.add_argument("--capacity-frac", type=float, default=0.03)
    ap.add_argument("--e2e-gb", type=float, default=10.0, help="host-resident state for the e2e leg (GB)")
    ap.add_argument("--cpu-elements", type=float, default=2.0e9, help="oracle sample size (elements)")
    ap.add_argument("--ref-elements", type=float, default=4e8, help="--impl reference: elements per step")
    ap.add_argument("--variant", default="mirror", choices=["mirror", "trainer"],
                    help="association of the generator's forward AdamW step (only changes the inputs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-codec", action="store_true", help="skip the storage-mediated path's legs")
    ap.add_argument("--probes", action="store_true",
                    help="time the memory-system probes (read-only stream, isolated sparse accesses) and exit")
    ap.add_argument("--no-extra-workloads", action="store_true",
                    help="skip the config 4 / config 1 / density-sweep legs that follow the headline workload")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    import paper_2608_00455_b200 as dte

    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if args.probes:
        if rank == 0:
            run_probes(device)
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    t_gen = time.time()
    workload = args.workload
    free_b, _ = torch.cuda.mem_get_info(device)
    if workload == "full" and free_b < 128e9:
        # the full state needs ~115 GB (98.3 GB of theta/m/v + 16.4 GB of shards + lists); on a
        # smaller or partly occupied GPU run as many layers as fit and say so in config.workload
        n_fit = max(1, int((free_b * 0.85 - 6e9) // (192946432 * 14.6)))
        workload = f"layers:{min(36, n_fit)}"
        log(f"[bench] only {free_b / 1e9:.0f} GB free: falling back to --workload {workload}")
    wl = build_workload(workload, device)
    wl.variant = args.variant
    plan = wl.plan
    st, shards = materialize_resident(wl, device, dte)
    torch.cuda.synchronize()
    log(f"[bench] generated {wl.name}: {plan.total_source_elements()} source elements in {time.time() - t_gen:.1f}s, "
        f"{torch.cuda.memory_allocated() / 1e9:.1f} GB allocated")

    lay = dte.Layout.from_plan(plan, local_rank)
    N = lay.num_elements
    delta = lay.new_delta(int(N * args.capacity_frac) + 1024)
    tabs = lay.source_tables(st.theta, st.m, st.v)
    shard_tab = lay.shard_table(shards)
    hp = wl.hp.as_args()
    stream = torch.cuda.current_stream()

    # ---- untimed first pass: reconstruction-based change set vs the true one ----------------
    dte.dte_extract_delta(lay, tabs, *hp, delta)
    torch.cuda.synchronize()
    bits = delta.status_bits()
    if bits:
        raise SystemExit(f"extract reported device status bits {bits} (capacity {delta.capacity}, total {delta.total()})")
    M = delta.total()
    broken = int(delta.counters[3].item())      # reconstructions that came out NaN or overflowed
    lp_d = delta.list_ptr.cpu()
    init_vals = torch.empty(M, dtype=torch.int16, device=device)
    for k in range(plan.n_shards):
        a, b = int(lp_d[k]), int(lp_d[k + 1])
        if b > a:
            init_vals[a:b] = shards[k][delta.offsets[a:b].to(torch.int64) & 0xFFFFFFFF]
    dte.dte_apply(lay, delta, shard_tab)
    torch.cuda.synchronize()
    fn = fp = None
    if rank == 0:
        fn, fp = reconstruction_vs_truth(plan, st, shards, init_vals, (lp_d, delta.offsets, delta.values))
    del init_vals
    log(f"[bench] N={N} changed={M} ({100.0 * M / N:.3f} %), FN={fn} FP={fp}")

    # ---- timed region -------------------------------------------------------------------------
    def step(ev=None):
        if ev: ev[0].record(stream)
        dte.dte_extract_delta(lay, tabs, *hp, delta)
        if ev: ev[1].record(stream)
        dte.dte_apply(lay, delta, shard_tab)
        if ev: ev[2].record(stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    flush = None
    if 12 * N < 2e9:      # the state could sit in the 126 MB L2: evict it between timed steps
        flush = torch.empty(1 << 28, dtype=torch.uint8, device=device)

    def timed_region():
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
            time.sleep(0.3)
        if dist: dist.barrier()
        torch.cuda.synchronize()
        w0 = time.time()
        for i in range(args.steps):
            if flush is not None:
                flush.zero_()
            step(evs[i])
        torch.cuda.synchronize()
        if dist: dist.barrier()
        w1 = time.time()
        return evs, (sampler.stop(w0, w1) if rank == 0 else None)

    evs, clocks = timed_region()
    # a timed region that saw a hardware or thermal slowdown is not a measurement: take it once more
    slow = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
    again = torch.tensor([int(bool(clocks and slow & set(clocks["reasons"])))], device=device)
    if dist: dist.broadcast(again, 0)
    if int(again.item()):
        first = clocks
        time.sleep(5.0)
        evs, clocks = timed_region()
        if clocks is not None:
            clocks["remeasured_after"] = first["reasons"]
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    if flush is not None:  # leave the flush writes out of the step time
        total_ms = sum(e[0].elapsed_time(e[2]) for e in evs)
    ext_ms = [e[0].elapsed_time(e[1]) for e in evs]
    app_ms = [e[1].elapsed_time(e[2]) for e in evs]
    n_lists = lay.num_lists
    launch_info = lay.last_launch()
    launches = (launch_info["kernels"] + 1) * args.steps     # extract call + apply, per step
    bytes_per_step = 12.0 * N + 6.0 * M
    total_ms, bytes_all = aggregate_over_ranks(total_ms, bytes_per_step, dist, device)
    ms_per_step = total_ms / args.steps
    value = bytes_all / (ms_per_step * 1e-3) / 1e9
    ext_avg = sum(ext_ms) / len(ext_ms)
    app_avg = sum(app_ms) / len(app_ms)
    apply_bpe = apply_traffic_per_entry()
    peak, peak_kind = measured_peak()
    achieved = bytes_per_step / (ext_avg * 1e-3) / 1e9
    traffic, traffic_src = extract_traffic(N)

    # ---- practical ceiling for a read-only kernel: plain streaming reads of the same tensors --------
    ceiling = None
    if rank == 0:
        ceiling = read_ceiling(device)
        log(f"[bench] read-only streaming ceiling: {ceiling}")

    # ---- same-cluster transfer fused into the extract (outside the timed step) --------------------
    push = None
    if rank == 0 and not args.no_codec:
        push = time_push(dte, lay, tabs, hp, delta, device)
        if push and "ms" in push:
            push["extra_ms_over_extract"] = push["ms"] - ext_avg
        log(f"[bench] push: {push}")

    # ---- storage path: chunk codec on the step's lists (outside the timed step) ------------------
    codec = None
    if rank == 0 and not args.no_codec:
        codec = time_storage_path(dte, wl, st, shards, hp, delta.capacity, device, peak)
        log(f"[bench] storage path: {codec}")

    # ---- end to end through the host-buffer entry point -----------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, wl, st, device, dte, world, dist)

    # ---- CPU baseline: the oracle on a bounded sample ---------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        chosen, n_el = oracle_sample(wl, st, int(args.cpu_elements))
        dt, res = time_oracle(wl, st, chosen)
        ops = plan.ops_array()
        ops = ops[np.isin(ops[:, 0], chosen)]
        scanned = int((ops[:, 4] * ops[:, 5]).sum())
        m_cpu = int(res[0][-1])
        # the sampled lists must equal the GPU's
        lp_g, off_g, val_g = delta.to_host()
        ok = True
        for k in sorted(set(int(x) for x in ops[:, 1])):
            full = all(int(o[0]) in chosen for o in plan.ops if o[1] == k)
            if not full:
                continue
            a, b, c, d = int(lp_g[k]), int(lp_g[k + 1]), int(res[0][k]), int(res[0][k + 1])
            ok &= (b - a == d - c) and np.array_equal(off_g[a:b], res[1][c:d]) and np.array_equal(val_g[a:b], res[2][c:d])
        cpu = {"value": (12.0 * scanned + 6.0 * m_cpu) / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {len(chosen)} source tensors ({scanned} scanned elements) of {wl.name}, extract only, "
                         f"{dt:.1f} s", "elements_per_s": scanned / dt, "lists_equal_gpu": bool(ok)}
        # the same oracle on every host core, disjoint tensors per thread
        k = os.cpu_count() or 1
        dt_k, scanned_k, m_k, used = time_oracle_threads(wl, st, chosen, k)
        cpu["all_cores"] = {"value": (12.0 * scanned_k + 6.0 * m_k) / dt_k / 1e9, "unit": UNIT, "cores": used,
                            "seconds": dt_k, "elements_per_s": scanned_k / dt_k,
                            "sample": "the same tensors, split over the threads largest first"}

    # ---- the other quoted workloads, one after the other on the freed GPU -------------------------
    extra = {}
    if rank == 0 and world == 1 and args.workload == "full" and not args.no_extra_workloads:
        import gc
        del st, shards, delta, tabs, shard_tab, lay
        gc.collect()
        torch.cuda.empty_cache()
        legs = max(10, min(args.steps, 30))
        t0 = time.time()
        extra["config4"] = time_leg(dte, lambda i: configs.config4(device), device, legs, args.warmup, peak, 0.04)
        log(f"[bench] config 4: {extra['config4']} ({time.time() - t0:.0f} s)")
        extra["config1"] = time_leg(dte, lambda i: configs.config1(seed=1234 + i), device, 48, args.warmup, peak, copies=8)
        log(f"[bench] config 1: {extra['config1']}")
        sweep = []
        for (lr, step_t, wd, sg) in density_sweep_points():
            r = time_leg(dte, lambda i: configs.config5(lr, step_t, wd, sg), device, 20, args.warmup, peak, 0.03)
            r["sigma_g"] = sg
            sweep.append(r)
            log(f"[bench] sweep lr={lr:g} sigma_g={sg:g}: rho={r.get('changed_frac')} extract {r.get('extract_GBps')} GB/s")
        extra["density_sweep"] = sweep

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "elements_scanned": N, "changed": M, "changed_frac": M / N,
                       "lists": n_lists, "l2": "inputs larger than L2 (no flush needed)" if flush is None else "256 MB written between timed steps to flush L2",
                       "hyper": {"step": wl.hp.step, "lr": wl.hp.lr, "wd": wl.hp.wd}, **wl.notes},
            "extract": {"ms": ext_avg, "ms_min": min(ext_ms), "ms_median": statistics.median(ext_ms), "GBps": achieved, "elements_per_s": N / (ext_avg * 1e-3),
                        "frac_of_8TBps": achieved / 8000.0},
            "apply": {"ms": app_avg, "ms_min": min(app_ms), "ms_median": statistics.median(app_ms),
                      "Mchanged_per_s": M / (app_avg * 1e-3) / 1e6,
                      "GBps_algorithmic": 8.0 * M / (app_avg * 1e-3) / 1e9,
                      # DRAM traffic per entry measured by ncu at this density (sector fill and
                      # write-back of every touched sector + the lists); model figure if no capture
                      "dram_bytes_per_entry": apply_bpe if apply_bpe else 70.0,
                      "dram_bytes_per_entry_source": os.path.basename(APPLY_TRAFFIC_JSON) if apply_bpe else "model: 32 B fill + 32 B write-back + 6 B list",
                      "GBps_dram_traffic": (apply_bpe or 70.0) * M / (app_avg * 1e-3) / 1e9,
                      "frac_of_peak_dram_traffic": (apply_bpe or 70.0) * M / (app_avg * 1e-3) / 1e9 / peak},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "traffic_source": traffic_src, "peak_source": peak_kind,
                         "kernel": "extract call (extract_kernel launches + scan + gather)",
                         "read_only_ceiling": ceiling,
                         "frac_of_read_only_ceiling": achieved / ceiling["GBps"] if ceiling else None},
            "reconstruction_vs_truth": {"false_negatives": fn, "false_positives": fp, "variant": wl.variant,
                                        "nan_or_overflowed_reconstructions": broken},
            "storage_path": codec, "push": push,
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "launch": launch_info, **extra,
        }
        print(json.dumps(out), flush=True)
    if dist:
        dist.destroy_process_group()


def run_e2e(args, wl, st, device, dte, world, dist):
    """Same metric through dte_extract_delta_host: pinned host theta/m/v -> device -> extract ->
    apply -> lists back to the host, copies inside the timed region."""
    plan = wl.plan
    budget = int(args.e2e_gb * 1e9 / 12)
    chosen, n = [], 0
    for p in range(plan.n_tensors):
        if n + plan.numel(p) > budget and chosen:
            break
        chosen.append(p); n += plan.numel(p)
    sub = plans.Plan()
    remap = {}
    for p in chosen:
        remap[p] = sub.add_tensor(plan.tensor_names[p], plan.tensor_shapes[p])
    kmap = {}
    for o in plan.ops:
        if o[0] in remap:
            if o[1] not in kmap:
                kmap[o[1]] = sub.add_shard(plan.shard_names[o[1]], plan.shard_receivers[o[1]], plan.shard_numels[o[1]])
            sub.ops.append((remap[o[0]], kmap[o[1]]) + tuple(o[2:]))
    lay = dte.Layout.from_plan(sub, device.index)
    th, mm, vv = ([lst[p].cpu().pin_memory() for p in chosen] for lst in (st.theta, st.m, st.v))
    ws = torch.empty(lay.host_workspace_bytes, dtype=torch.uint8, device=device)
    N = lay.num_elements
    delta = lay.new_delta(int(N * args.capacity_frac) + 1024)
    res = dte.HostResult(lay.num_lists, delta.capacity)
    shards = [torch.zeros(nn, dtype=torch.int16, device=device) for nn in sub.shard_numels]
    tab = lay.shard_table(shards)
    hp = wl.hp.as_args()
    stream = torch.cuda.current_stream()

    def step():
        dte.dte_extract_delta_host(lay, th, mm, vv, *hp, ws, delta, res)
        dte.dte_apply(lay, delta, tab)

    for _ in range(2):
        step()
    torch.cuda.synchronize()
    steps = max(2, min(args.steps, 5))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist: dist.barrier()
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    M = int(res.counters[0])
    ms, bytes_all = aggregate_over_ranks(ms, 12.0 * N + 6.0 * M, dist, device)
    h2d = 12 * sub.total_source_elements()
    d2h = 6 * M + 8 * (lay.num_lists + 1) + 32
    return {"value": bytes_all / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "workload": f"first {len(chosen)} source tensors of {wl.name} held in pinned host memory "
                        f"({N} scanned elements); PCIe-bound"}


if __name__ == "__main__":
    main()
