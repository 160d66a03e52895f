"""Transfer-plan builders for the synthetic workloads (inputs only).

A plan is the paper's precomputed table T of hyper-rectangular overlaps
(Section 4.2.2): source tensors in the canonical training-side space, flat
receiver-local destination tensors ("shards"), and one operation per overlap.
This module only *describes* layouts; it evaluates none of the method's
arithmetic and is used by the tests, the benchmark, the CUDA binding's callers
and the oracle's callers alike.

Operation row (10 integers):
    src_tensor, dst_shard, a_s0, a_s1, e0, e1, dst_base, dst_ld, a_r0, a_r1
meaning: source coordinate u with a_s <= u < a_s + e lands at receiver flat
index  dst_base + (u0 - a_s0 + a_r0) * dst_ld + (u1 - a_s1 + a_r1).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import numpy as np


@dataclass
class Plan:
    tensor_names: List[str] = field(default_factory=list)
    tensor_shapes: List[Tuple[int, int]] = field(default_factory=list)
    shard_names: List[str] = field(default_factory=list)
    shard_receivers: List[int] = field(default_factory=list)
    shard_numels: List[int] = field(default_factory=list)
    ops: List[Tuple[int, ...]] = field(default_factory=list)
    # distributed-optimizer plans: flat element range [lo, hi) each source tensor's owner holds
    slice_ranges: List[Tuple[int, int]] = field(default_factory=list)

    @property
    def n_tensors(self) -> int:
        return len(self.tensor_shapes)

    @property
    def n_shards(self) -> int:
        return len(self.shard_numels)

    def ops_array(self) -> np.ndarray:
        return np.asarray(self.ops, dtype=np.int64).reshape(-1, 10)

    def numel(self, p: int) -> int:
        return self.tensor_shapes[p][0] * self.tensor_shapes[p][1]

    def total_source_elements(self) -> int:
        return sum(self.numel(p) for p in range(self.n_tensors))

    def total_scanned_elements(self) -> int:
        """Elements visited by a scan of every operation (replicas count once each)."""
        return int(sum(int(o[4]) * int(o[5]) for o in self.ops))

    # ---- primitives -------------------------------------------------------
    def add_tensor(self, name: str, shape: Sequence[int]) -> int:
        shape = tuple(int(s) for s in shape)
        if len(shape) == 1:
            shape = (shape[0], 1)
        assert len(shape) == 2
        self.tensor_names.append(name)
        self.tensor_shapes.append(shape)
        return len(self.tensor_shapes) - 1

    def add_shard(self, name: str, receiver: int, numel: int) -> int:
        self.shard_names.append(name)
        self.shard_receivers.append(int(receiver))
        self.shard_numels.append(int(numel))
        return len(self.shard_numels) - 1

    def add_op(self, src, dst, a_s, e, dst_base, dst_ld, a_r) -> None:
        self.ops.append((int(src), int(dst), int(a_s[0]), int(a_s[1]), int(e[0]), int(e[1]),
                         int(dst_base), int(dst_ld), int(a_r[0]), int(a_r[1])))

    # ---- rules (receiver r of R) -----------------------------------------
    def replicated(self, name: str, src: int, r: int) -> int:
        n0, n1 = self.tensor_shapes[src]
        k = self.add_shard(f"r{r}.{name}", r, n0 * n1)
        self.add_op(src, k, (0, 0), (n0, n1), 0, n1, (0, 0))
        return k

    def fused_rows(self, name: str, srcs: Sequence[int], r: int, R: int) -> int:
        """Row blocks [r*O_i/R, (r+1)*O_i/R) of each source, concatenated along rows.

        One source: column-parallel / vocab-parallel.  Three sources (q, k, v):
        fused qkv_proj split by head.  Two (gate, up): fused gate_up_proj.
        """
        cols = self.tensor_shapes[srcs[0]][1]
        rows = []
        for s in srcs:
            n0, n1 = self.tensor_shapes[s]
            assert n1 == cols and n0 % R == 0
            rows.append(n0 // R)
        k = self.add_shard(f"r{r}.{name}", r, sum(rows) * cols)
        at = 0
        for s, nr in zip(srcs, rows):
            self.add_op(s, k, (r * nr, 0), (nr, cols), 0, cols, (at, 0))
            at += nr
        return k

    def fused_qkv(self, name: str, q: int, k: int, v: int, r: int, R: int, hkv: int, hd: int) -> int:
        """Fused qkv_proj of receiver r split by head.  With R <= hkv every receiver takes
        hkv/R KV heads (plain row blocks).  With R > hkv (R a multiple of hkv) the KV heads are
        replicated: receiver r holds KV head r // (R / hkv) whole, next to its own Q heads, so
        R / hkv receivers emit the same K and V entries."""
        if hkv % R == 0:
            return self.fused_rows(name, [q, k, v], r, R)
        assert R % hkv == 0, "receivers must be a multiple of the KV heads to replicate them"
        cols = self.tensor_shapes[q][1]
        q_rows = self.tensor_shapes[q][0]
        assert q_rows % R == 0 and self.tensor_shapes[k] == (hkv * hd, cols) == self.tensor_shapes[v]
        nq = q_rows // R
        j = r // (R // hkv)
        dst = self.add_shard(f"r{r}.{name}", r, (nq + 2 * hd) * cols)
        self.add_op(q, dst, (r * nq, 0), (nq, cols), 0, cols, (0, 0))
        self.add_op(k, dst, (j * hd, 0), (hd, cols), 0, cols, (nq, 0))
        self.add_op(v, dst, (j * hd, 0), (hd, cols), 0, cols, (nq + hd, 0))
        return dst

    def row_parallel(self, name: str, src: int, r: int, R: int) -> int:
        """Column block [r*I/R, (r+1)*I/R) of the source (o_proj, down_proj)."""
        n0, n1 = self.tensor_shapes[src]
        assert n1 % R == 0
        w = n1 // R
        k = self.add_shard(f"r{r}.{name}", r, n0 * w)
        self.add_op(src, k, (0, r * w), (n0, w), 0, w, (0, 0))
        return k

    def expert_stack(self, name: str, per_expert_srcs: Sequence[Sequence[int]], r: int,
                     row_part: Tuple[int, int] = (0, 1), col_part: Tuple[int, int] = (0, 1)) -> int:
        """Stacked local experts: dst[l] = row-concatenation of per_expert_srcs[l].

        With expert tensor parallelism each source contributes only its row block
        row_part = (i, n) (w13: gate and up split along the intermediate dimension) or its
        column block col_part = (i, n) (w2: down_proj split along its input dimension)."""
        (ri, rn), (ci, cn) = row_part, col_part
        n1_full = self.tensor_shapes[per_expert_srcs[0][0]][1]
        assert n1_full % cn == 0
        cols = n1_full // cn
        rows_per = 0
        for s in per_expert_srcs[0]:
            assert self.tensor_shapes[s][0] % rn == 0
            rows_per += self.tensor_shapes[s][0] // rn
        k = self.add_shard(f"r{r}.{name}", r, len(per_expert_srcs) * rows_per * cols)
        for l, srcs in enumerate(per_expert_srcs):
            at = 0
            for s in srcs:
                n0, n1 = self.tensor_shapes[s]
                assert n1 == n1_full
                nr = n0 // rn
                self.add_op(s, k, (ri * nr, ci * cols), (nr, cols), l * rows_per * cols, cols, (at, 0))
                at += nr
            assert at == rows_per
        return k


# ---- model-shaped plans ------------------------------------------------------

def single_matrix_plan(rows=4096, cols=4096, tp=2) -> Plan:
    """One q_proj-shaped matrix, column-parallel over `tp` receivers."""
    p = Plan()
    w = p.add_tensor("q_proj", (rows, cols))
    for r in range(tp):
        p.fused_rows("q_proj", [w], r, tp)
    return p


QWEN3_8B = dict(hidden=4096, q_heads=32, kv_heads=8, head_dim=128, inter=12288, vocab=151936,
                layers=36)
QWEN3_30B_A3B = dict(hidden=2048, q_heads=32, kv_heads=4, head_dim=128, experts=128,
                     moe_inter=768, layers=48)


def _dense_layer_tensors(p: Plan, pre: str, d: dict) -> dict:
    h, hd = d["hidden"], d["head_dim"]
    t = {}
    t["q"] = p.add_tensor(pre + "q_proj", (d["q_heads"] * hd, h))
    t["k"] = p.add_tensor(pre + "k_proj", (d["kv_heads"] * hd, h))
    t["v"] = p.add_tensor(pre + "v_proj", (d["kv_heads"] * hd, h))
    t["o"] = p.add_tensor(pre + "o_proj", (h, d["q_heads"] * hd))
    t["gate"] = p.add_tensor(pre + "gate_proj", (d["inter"], h))
    t["up"] = p.add_tensor(pre + "up_proj", (d["inter"], h))
    t["down"] = p.add_tensor(pre + "down_proj", (h, d["inter"]))
    t["q_norm"] = p.add_tensor(pre + "q_norm", (hd,))
    t["k_norm"] = p.add_tensor(pre + "k_norm", (hd,))
    t["ln1"] = p.add_tensor(pre + "input_layernorm", (h,))
    t["ln2"] = p.add_tensor(pre + "post_attention_layernorm", (h,))
    return t


def _dense_layer_shards(p: Plan, pre: str, t: dict, r: int, R: int, d: dict) -> None:
    p.fused_qkv(pre + "qkv_proj", t["q"], t["k"], t["v"], r, R, d["kv_heads"], d["head_dim"])
    p.row_parallel(pre + "o_proj", t["o"], r, R)
    p.fused_rows(pre + "gate_up_proj", [t["gate"], t["up"]], r, R)
    p.row_parallel(pre + "down_proj", t["down"], r, R)
    for n in ("q_norm", "k_norm", "ln1", "ln2"):
        p.replicated(pre + n, t[n], r)


def qwen3_dense_plan(n_layers: int, tp: int, with_embeddings: bool, dims: dict = QWEN3_8B) -> Plan:
    """Qwen3-8B-shaped layers (+ embed_tokens / lm_head, vocab-parallel).

    Shards are numbered receiver-major, so one receiver's lists are adjacent
    in the concatenated output.
    """
    p = Plan()
    layers = [_dense_layer_tensors(p, f"layers.{l}.", dims) for l in range(n_layers)]
    emb = head = None
    if with_embeddings:
        emb = p.add_tensor("embed_tokens", (dims["vocab"], dims["hidden"]))
        head = p.add_tensor("lm_head", (dims["vocab"], dims["hidden"]))
    for r in range(tp):
        for l, t in enumerate(layers):
            _dense_layer_shards(p, f"layers.{l}.", t, r, tp, dims)
        if with_embeddings:
            p.fused_rows("embed_tokens", [emb], r, tp)
            p.fused_rows("lm_head", [head], r, tp)
    return p


def qwen3_moe_plan(n_layers: int, tp: int = 4, ep: int = 4, dims: dict = QWEN3_30B_A3B) -> Plan:
    """Qwen3-30B-A3B-shaped layers: attention TP, experts EP (stacked w13 / w2).

    One receiver set of `tp` ranks.  With ep < tp the experts are also tensor-parallel: the
    tp / ep ranks of an expert-parallel group split every local expert (gate and up by rows,
    down by columns).  With tp above the KV head count the KV heads are replicated."""
    assert tp % ep == 0, "receiver r holds TP rank r, EP rank r // (tp/ep), expert-TP rank r % (tp/ep)"
    etp = tp // ep
    p = Plan()
    h, hd, E, F = dims["hidden"], dims["head_dim"], dims["experts"], dims["moe_inter"]
    layers = []
    for l in range(n_layers):
        pre = f"layers.{l}."
        t = {}
        t["q"] = p.add_tensor(pre + "q_proj", (dims["q_heads"] * hd, h))
        t["k"] = p.add_tensor(pre + "k_proj", (dims["kv_heads"] * hd, h))
        t["v"] = p.add_tensor(pre + "v_proj", (dims["kv_heads"] * hd, h))
        t["o"] = p.add_tensor(pre + "o_proj", (h, dims["q_heads"] * hd))
        t["router"] = p.add_tensor(pre + "router", (E, h))
        t["q_norm"] = p.add_tensor(pre + "q_norm", (hd,))
        t["k_norm"] = p.add_tensor(pre + "k_norm", (hd,))
        t["ln1"] = p.add_tensor(pre + "input_layernorm", (h,))
        t["ln2"] = p.add_tensor(pre + "post_attention_layernorm", (h,))
        t["experts"] = []
        for e in range(E):
            g = p.add_tensor(pre + f"experts.{e}.gate_proj", (F, h))
            u = p.add_tensor(pre + f"experts.{e}.up_proj", (F, h))
            dn = p.add_tensor(pre + f"experts.{e}.down_proj", (h, F))
            t["experts"].append((g, u, dn))
        layers.append(t)
    e_loc = E // ep
    for r in range(tp):
        for l, t in enumerate(layers):
            pre = f"layers.{l}."
            p.fused_qkv(pre + "qkv_proj", t["q"], t["k"], t["v"], r, tp, dims["kv_heads"], hd)
            p.row_parallel(pre + "o_proj", t["o"], r, tp)
            for n in ("router", "q_norm", "k_norm", "ln1", "ln2"):
                p.replicated(pre + n, t[n], r)
            g_ep, g_tp = r // etp, r % etp
            mine = t["experts"][g_ep * e_loc:(g_ep + 1) * e_loc]
            p.expert_stack(pre + "w13", [(g, u) for g, u, _ in mine], r, row_part=(g_tp, etp))
            p.expert_stack(pre + "w2", [(dn,) for _, _, dn in mine], r, col_part=(g_tp, etp))
    return p


# ---- dense evaluation of a plan with tensor slicing --------------------------

def scatter_dense(plan: Plan, dense_by_tensor, shards) -> None:
    """Copy every source tensor's overlap regions into the flat shard buffers.

    `dense_by_tensor[p]` is a 2-D (or 1-D) torch tensor of the shard dtype and
    `shards[k]` a flat torch tensor of numel shard_numels[k].  Pure strided
    copies (the dense meaning of the operation table); used to initialise
    receiver buffers and to build expected end states.
    """
    for (src, dst, a0, a1, e0, e1, base, ld, r0, r1) in plan.ops:
        s = dense_by_tensor[src]
        if s is None:
            continue
        s2 = s.reshape(plan.tensor_shapes[src])
        view = shards[dst].as_strided((e0, e1), (ld, 1), base + r0 * ld + r1)
        view.copy_(s2[a0:a0 + e0, a1:a1 + e1])


# ---- Megatron-Core-native training-side layouts -------------------------------------------------
#
# Source tensors in the trainer's own organisation (Appendix B of the paper): per sender TP rank a
# fused, GQA-interleaved linear_qkv shard [Q_{jg..(j+1)g-1}, K_j, V_j] per kv group j (Eq. 14-16), a
# fused linear_fc1 shard [gate_s; up_s], column shards of linear_proj / linear_fc2, vocab shards
# of the embeddings, and - with a distributed optimizer - every such shard cut into `dp`
# contiguous flat slices, each owned by one data-parallel rank.  The receiver side is unchanged.

def restrict_to_flat_range(op, n1: int, lo: int, hi: int):
    """The parts of operation `op` whose source elements lie in the flat range [lo, hi) of a
    row-major source with n1 columns: at most a partial first row, whole middle rows and a
    partial last row (each a legal operation: whole destination rows or one row)."""
    src, dst, a0, a1, e0, e1, base, ld, r0, r1 = op
    out = []

    def emit(row_lo, row_hi, col_lo, col_hi):
        row_lo, row_hi = max(row_lo, a0), min(row_hi, a0 + e0)
        col_lo, col_hi = max(col_lo, a1), min(col_hi, a1 + e1)
        if row_lo >= row_hi or col_lo >= col_hi:
            return
        if col_lo == a1 and col_hi == a1 + e1:          # the operation's full width: keep rows together
            out.append((src, dst, row_lo, a1, row_hi - row_lo, e1, base, ld, r0 + row_lo - a0, r1))
        else:                                            # partial width: one operation per row
            for row in range(row_lo, row_hi):
                out.append((src, dst, row, col_lo, 1, col_hi - col_lo, base, ld, r0 + row - a0,
                            r1 + col_lo - a1))

    first_full = -(-lo // n1)
    last_full = hi // n1
    if first_full > last_full:                           # the range lies inside one row
        emit(lo // n1, lo // n1 + 1, lo % n1, hi - (lo // n1) * n1)
        return out
    if lo % n1:
        emit(lo // n1, lo // n1 + 1, lo % n1, n1)
    emit(first_full, last_full, 0, n1)
    if hi % n1:
        emit(last_full, last_full + 1, 0, hi % n1)
    return out


def _overlap(lo_a, hi_a, lo_b, hi_b):
    lo, hi = max(lo_a, lo_b), min(hi_a, hi_b)
    return (lo, hi) if lo < hi else None


def mcore_dense_plan(n_layers: int, tp_send: int, tp_recv: int, with_embeddings: bool,
                     dims: dict = QWEN3_8B, dp: int = 1, align: int = 4) -> Plan:
    """Qwen3-dense layers with Megatron-Core-native sources (see above) and the usual receivers.

    Column-split tensors (linear_proj, linear_fc2) map with whole destination rows when the
    receiver shard lies inside one sender shard (tp_send divides tp_recv); otherwise the
    builder falls back to one operation per destination row piece.
    """
    P_, R = tp_send, tp_recv
    h, hd, hq, hkv, F = dims["hidden"], dims["head_dim"], dims["q_heads"], dims["kv_heads"], dims["inter"]
    g = hq // hkv
    assert hkv % P_ == 0 and hkv % R == 0 and F % P_ == 0 and F % R == 0
    p = Plan()
    raw_ops = []       # operations before the data-parallel cut, with the source's column count

    srcs = {}          # (layer, kind, sender) -> tensor index
    for l in range(n_layers):
        pre = f"layers.{l}."
        for s in range(P_):
            srcs[l, "qkv", s] = p.add_tensor(f"{pre}linear_qkv.tp{s}", ((hq + 2 * hkv) * hd // P_, h))
            srcs[l, "proj", s] = p.add_tensor(f"{pre}linear_proj.tp{s}", (h, hq * hd // P_))
            srcs[l, "fc1", s] = p.add_tensor(f"{pre}linear_fc1.tp{s}", (2 * F // P_, h))
            srcs[l, "fc2", s] = p.add_tensor(f"{pre}linear_fc2.tp{s}", (h, F // P_))
        for n, shape in (("q_norm", (hd,)), ("k_norm", (hd,)), ("input_layernorm", (h,)),
                         ("post_attention_layernorm", (h,))):
            srcs[l, n, 0] = p.add_tensor(pre + n, shape)      # replicated on senders: rank 0's copy is used
    if with_embeddings:
        V = dims["vocab"]
        assert V % P_ == 0 and V % R == 0
        for s in range(P_):
            srcs["emb", s] = p.add_tensor(f"embed_tokens.tp{s}", (V // P_, h))
            srcs["head", s] = p.add_tensor(f"lm_head.tp{s}", (V // P_, h))

    def add(src, dst, a_s, e, base, ld, a_r):
        raw_ops.append((int(src), int(dst), int(a_s[0]), int(a_s[1]), int(e[0]), int(e[1]), int(base),
                        int(ld), int(a_r[0]), int(a_r[1])))

    def row_split(dst, dst_row0, dst_cols, kind_key, total_rows, want_lo, want_hi):
        """Rows [want_lo, want_hi) of a logical [total_rows, cols] tensor whose sender s holds rows
        [s*total/P, (s+1)*total/P) -> destination rows starting at dst_row0."""
        per = total_rows // P_
        for s in range(P_):
            ov = _overlap(want_lo, want_hi, s * per, (s + 1) * per)
            if ov:
                add(srcs[kind_key(s)], dst, (ov[0] - s * per, 0), (ov[1] - ov[0], dst_cols), 0, dst_cols,
                    (dst_row0 + ov[0] - want_lo, 0))

    def col_split(dst, kind_key, rows, total_cols, want_lo, want_hi):
        per = total_cols // P_
        w = want_hi - want_lo
        for s in range(P_):
            ov = _overlap(want_lo, want_hi, s * per, (s + 1) * per)
            if not ov:
                continue
            if ov[1] - ov[0] == w:      # whole destination rows
                add(srcs[kind_key(s)], dst, (0, ov[0] - s * per), (rows, w), 0, w, (0, 0))
            else:                       # a piece of every destination row: one operation per row
                for row in range(rows):
                    add(srcs[kind_key(s)], dst, (row, ov[0] - s * per), (1, ov[1] - ov[0]), 0, w,
                        (row, ov[0] - want_lo))

    for r in range(R):
        for l in range(n_layers):
            pre = f"layers.{l}."
            # fused qkv_proj by head: kv groups [r*hkv/R, (r+1)*hkv/R)
            q_rows, kv_rows = hq * hd // R, hkv * hd // R
            k = p.add_shard(f"r{r}.{pre}qkv_proj", r, (q_rows + 2 * kv_rows) * h)
            for j in range(r * hkv // R, (r + 1) * hkv // R):
                s, jl, jr = j // (hkv // P_), j % (hkv // P_), j - r * hkv // R
                src = srcs[l, "qkv", s]
                blk = jl * (g + 2) * hd                                   # Eq. 14: [Q x g, K, V] per group
                add(src, k, (blk, 0), (g * hd, h), 0, h, (jr * g * hd, 0))
                add(src, k, (blk + g * hd, 0), (hd, h), 0, h, (q_rows + jr * hd, 0))
                add(src, k, (blk + (g + 1) * hd, 0), (hd, h), 0, h, (q_rows + kv_rows + jr * hd, 0))
            C = hq * hd
            k = p.add_shard(f"r{r}.{pre}o_proj", r, h * C // R)
            col_split(k, lambda s: (l, "proj", s), h, C, r * C // R, (r + 1) * C // R)
            # fused gate_up_proj: gate rows [r*F/R, ...) then up rows; sender s holds [gate_s; up_s]
            k = p.add_shard(f"r{r}.{pre}gate_up_proj", r, 2 * F // R * h)
            per = F // P_
            for half in range(2):                                         # 0 = gate, 1 = up
                for s in range(P_):
                    ov = _overlap(r * F // R, (r + 1) * F // R, s * per, (s + 1) * per)
                    if ov:
                        add(srcs[l, "fc1", s], k, (half * per + ov[0] - s * per, 0), (ov[1] - ov[0], h), 0, h,
                            (half * F // R + ov[0] - r * F // R, 0))
            k = p.add_shard(f"r{r}.{pre}down_proj", r, h * F // R)
            col_split(k, lambda s: (l, "fc2", s), h, F, r * F // R, (r + 1) * F // R)
            for n in ("q_norm", "k_norm", "input_layernorm", "post_attention_layernorm"):
                src = srcs[l, n, 0]
                n0 = p.tensor_shapes[src][0]
                k = p.add_shard(f"r{r}.{pre}{n}", r, n0)
                add(src, k, (0, 0), (n0, 1), 0, 1, (0, 0))
        if with_embeddings:
            V = dims["vocab"]
            for name, key in (("embed_tokens", "emb"), ("lm_head", "head")):
                k = p.add_shard(f"r{r}.{name}", r, V // R * h)
                row_split(k, 0, h, lambda s, key=key: (key, s), V, r * V // R, (r + 1) * V // R)

    if dp == 1:
        p.ops = raw_ops
        return p
    # distributed optimizer: every source tensor is cut into `dp` flat slices (boundaries on
    # multiples of `align` elements); slice d becomes its own source tensor of the same shape
    q = Plan(shard_names=p.shard_names, shard_receivers=p.shard_receivers, shard_numels=p.shard_numels)
    new_index = {}
    for t, (name, shape) in enumerate(zip(p.tensor_names, p.tensor_shapes)):
        n = shape[0] * shape[1]
        cuts = [min(n, -(-(n * d // dp) // align) * align) for d in range(dp)] + [n]
        for d in range(dp):
            new_index[t, d] = q.add_tensor(f"{name}.dp{d}", shape)
            q.slice_ranges.append((cuts[d], cuts[d + 1]))
    for op in raw_ops:
        n1 = p.tensor_shapes[op[0]][1]
        for d in range(dp):
            lo, hi = q.slice_ranges[new_index[op[0], d]]
            for piece in restrict_to_flat_range(op, n1, lo, hi):
                q.ops.append((new_index[op[0], d],) + tuple(piece[1:]))
    return q


def canonical_plan(names: Sequence[str], shapes: Sequence[Sequence[int]]) -> Plan:
    """Identity plan: every source tensor maps onto one destination of its own shape, so the
    lists are the canonical (index, value) pairs of Eq. 4 - what the storage path publishes
    before any receiver layout is applied (Section 4.4)."""
    p = Plan()
    for name, shape in zip(names, shapes):
        t = p.add_tensor(name, shape)
        p.replicated(name, t, 0)
    return p


def tensor_senders(plan: Plan, tp_send: int, dp: int = 1) -> List[int]:
    """Sender index of every source tensor of a Megatron-Core-native plan, from its name:
    `.tp{s}` shards belong to TP rank s, `.dp{d}` slices to data-parallel rank d, tensors
    replicated over TP ranks are taken from TP rank 0.  Sender index = s * dp + d."""
    import re
    out = []
    for name in plan.tensor_names:
        s = re.search(r"\.tp(\d+)", name)
        d = re.search(r"\.dp(\d+)", name)
        s, d = int(s.group(1)) if s else 0, int(d.group(1)) if d else 0
        assert s < tp_send and d < dp
        out.append(s * dp + d)
    return out


def sender_subplan(plan: Plan, owners: Sequence[int], sender: int) -> Plan:
    """The plan as sender `sender` executes it: every tensor and shard keeps its index, only the
    operations whose source tensor the sender owns remain (in plan order)."""
    q = Plan(tensor_names=plan.tensor_names, tensor_shapes=plan.tensor_shapes, shard_names=plan.shard_names,
             shard_receivers=plan.shard_receivers, shard_numels=plan.shard_numels)
    q.slice_ranges = plan.slice_ranges
    q.ops = [op for op in plan.ops if owners[op[0]] == sender]
    return q


def random_plan(seed: int, max_tensors: int = 6) -> Plan:
    """A seeded plan of arbitrary hyper-rectangles for parity fuzzing: odd shapes, row / column /
    grid splits, single-row pieces assembled into wider destination rows, stacked destinations
    with gaps, replication, regions and whole tensors no operation reads.  Every destination
    region is a contiguous flat range and no two overlap (the layout's rules)."""
    rng = np.random.default_rng(seed)
    p = Plan()

    def cuts(n, k):
        """k random consecutive blocks covering [0, n)."""
        k = max(1, min(k, n))
        inner = np.sort(rng.choice(np.arange(1, n), size=k - 1, replace=False)) if k > 1 else np.zeros(0, np.int64)
        b = [0] + [int(x) for x in inner] + [n]
        return list(zip(b[:-1], b[1:]))

    n_t = int(rng.integers(1, max_tensors + 1))
    for t in range(n_t):
        if rng.random() < 0.25:
            shape = (int(rng.integers(1, 60000)), 1)
        else:
            shape = (int(rng.integers(1, 400)), int(rng.integers(1, 900)))
        src = p.add_tensor(f"t{t}", shape)
        n0, n1 = shape
        kind = rng.choice(["rows", "cols", "grid", "replicate", "row_pieces", "stack", "skip"],
                          p=[0.2, 0.2, 0.15, 0.1, 0.15, 0.15, 0.05])
        recv = lambda: int(rng.integers(0, 4))
        if kind == "skip":
            continue
        if kind == "rows":                    # row blocks, each its own destination (some dropped)
            for lo, hi in cuts(n0, int(rng.integers(1, 5))):
                if rng.random() < 0.15:
                    continue
                k = p.add_shard(f"t{t}.rows{lo}", recv(), (hi - lo) * n1)
                p.add_op(src, k, (lo, 0), (hi - lo, n1), 0, n1, (0, 0))
        elif kind == "cols":                  # column blocks: strided sources, whole destination rows
            for lo, hi in cuts(n1, int(rng.integers(1, 5))):
                k = p.add_shard(f"t{t}.cols{lo}", recv(), n0 * (hi - lo))
                p.add_op(src, k, (0, lo), (n0, hi - lo), 0, hi - lo, (0, 0))
        elif kind == "grid":
            for r0, r1 in cuts(n0, int(rng.integers(1, 4))):
                for c0, c1 in cuts(n1, int(rng.integers(1, 4))):
                    k = p.add_shard(f"t{t}.g{r0}.{c0}", recv(), (r1 - r0) * (c1 - c0))
                    p.add_op(src, k, (r0, c0), (r1 - r0, c1 - c0), 0, c1 - c0, (0, 0))
        elif kind == "replicate":
            for r in range(int(rng.integers(2, 5))):
                k = p.add_shard(f"t{t}.copy{r}", r, n0 * n1)
                p.add_op(src, k, (0, 0), (n0, n1), 0, n1, (0, 0))
        elif kind == "row_pieces":            # destination rows wider than the pieces that fill them
            rows = min(n0, int(rng.integers(1, 12)))
            pad_l, pad_r = int(rng.integers(0, 9)), int(rng.integers(0, 9))
            ld = pad_l + n1 + pad_r
            k = p.add_shard(f"t{t}.pieces", recv(), rows * ld)
            for row in range(rows):
                for c0, c1 in cuts(n1, int(rng.integers(1, 4))):
                    if rng.random() < 0.1:
                        continue              # a hole inside the destination row
                    p.add_op(src, k, (row, c0), (1, c1 - c0), 0, ld, (row, pad_l + c0))
        else:                                 # stack: row blocks at scattered bases of one destination
            blocks = cuts(n0, int(rng.integers(1, 5)))
            order = rng.permutation(len(blocks))
            gap = int(rng.integers(0, 3)) * int(rng.integers(0, 50))
            base, places = 0, {}
            for i in order:
                lo, hi = blocks[int(i)]
                places[int(i)] = base
                base += (hi - lo) * n1 + gap
            k = p.add_shard(f"t{t}.stack", recv(), base + int(rng.integers(0, 20)))
            for i, (lo, hi) in enumerate(blocks):
                p.add_op(src, k, (lo, 0), (hi - lo, n1), places[i], n1, (0, 0))
    if not p.ops:                             # never hand out an empty plan
        k = p.add_shard("t0.all", 0, p.numel(0))
        p.add_op(0, k, (0, 0), p.tensor_shapes[0], 0, p.tensor_shapes[0][1], (0, 0))
    return p
