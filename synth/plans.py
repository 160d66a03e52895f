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

    def row_parallel(self, name: str, src: int, r: int, R: int) -> int:
        """Column block [r*I/R, (r+1)*I/R) of the source (o_proj, down_proj)."""
        n0, n1 = self.tensor_shapes[src]
        assert n1 % R == 0
        w = n1 // R
        k = self.add_shard(f"r{r}.{name}", r, n0 * w)
        self.add_op(src, k, (0, r * w), (n0, w), 0, w, (0, 0))
        return k

    def expert_stack(self, name: str, per_expert_srcs: Sequence[Sequence[int]], r: int) -> int:
        """Stacked local experts: dst[l] = row-concatenation of per_expert_srcs[l]."""
        cols = self.tensor_shapes[per_expert_srcs[0][0]][1]
        rows_per = sum(self.tensor_shapes[s][0] for s in per_expert_srcs[0])
        k = self.add_shard(f"r{r}.{name}", r, len(per_expert_srcs) * rows_per * cols)
        for l, srcs in enumerate(per_expert_srcs):
            at = 0
            for s in srcs:
                n0, n1 = self.tensor_shapes[s]
                assert n1 == cols
                self.add_op(s, k, (0, 0), (n0, n1), l * rows_per * cols, cols, (at, 0))
                at += n0
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


def _dense_layer_shards(p: Plan, pre: str, t: dict, r: int, R: int) -> None:
    p.fused_rows(pre + "qkv_proj", [t["q"], t["k"], t["v"]], r, R)
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
            _dense_layer_shards(p, f"layers.{l}.", t, r, tp)
        if with_embeddings:
            p.fused_rows("embed_tokens", [emb], r, tp)
            p.fused_rows("lm_head", [head], r, tp)
    return p


def qwen3_moe_plan(n_layers: int, tp: int = 4, ep: int = 4, dims: dict = QWEN3_30B_A3B) -> Plan:
    """Qwen3-30B-A3B-shaped layers: attention TP, experts EP (stacked w13 / w2)."""
    assert tp == ep, "one receiver set: receiver r holds TP rank r and EP rank r"
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
            p.fused_rows(pre + "qkv_proj", [t["q"], t["k"], t["v"]], r, tp)
            p.row_parallel(pre + "o_proj", t["o"], r, tp)
            for n in ("router", "q_norm", "k_norm", "ln1", "ln2"):
                p.replicated(pre + n, t[n], r)
            mine = t["experts"][r * e_loc:(r + 1) * e_loc]
            p.expert_stack(pre + "w13", [(g, u) for g, u, _ in mine], r)
            p.expert_stack(pre + "w2", [(dn,) for _, _, dn in mine], r)
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
