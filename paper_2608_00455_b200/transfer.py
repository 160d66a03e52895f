"""Two-round same-cluster delta transfer (Section 4.3) over torch.distributed point-to-point calls.

The transfer plan fixes, before any data exists, which sender feeds which receiver and in which
order; only the entry counts c_o vary from version to version, and they may be zero.  Round 1
therefore moves, for every (sender, receiver) pair of the plan, the counts of ALL of the pair's
operations in plan order, zeros included; the receiver sizes its buffers from them.  Round 2 moves
the indices I_o and the values V_o.  Because both sides derive the same schedule from the plan and
never drop a call on one side only, the point-to-point calls stay matched.

What is B200-specific here is only the shape of the messages: the extract kernel emits the lists
of one receiver back to back (shards are grouped by receiver), in destination order, so the whole
payload for a receiver is ONE contiguous slice of the extract output - it is sent as it lies in
HBM, without packing - and the per-operation payloads (I_o, V_o) are consecutive runs of that
slice whose lengths are the c_o of round 1.  All calls of a round are issued as one batch (NCCL
groups them), so no ordering between pairs can deadlock.

This module is plumbing: it holds no arithmetic of the method and launches no kernel.  Tensors may
live on any device the process group's backend supports (NCCL: CUDA, gloo: CPU).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist


@dataclass
class Route:
    """One (sender, receiver) pair of the plan."""
    sender: int                 # sender index (training side)
    receiver: int               # receiver index (inference side)
    ops: np.ndarray             # operations of the pair (indices into the whole plan), plan order
    local_ops: np.ndarray       # the same operations as positions in the sender's own operation list
    op_slot: np.ndarray         # for each of them, the position of its shard in `shards`
    shards: np.ndarray          # shard ids of the receiver, ascending (one list each)
    contiguous: bool            # the shards are consecutive: the payload is one slice


@dataclass
class Received:
    """What a receiver holds after both rounds, for one sender."""
    sender: int
    op_counts: np.ndarray       # c_o of the route's operations, plan order
    list_ptr: np.ndarray        # uint64[n_shards + 1] over ALL shards of the plan (zeros elsewhere)
    offsets: torch.Tensor       # int32 bit patterns of the uint32 receiver-local offsets
    values: torch.Tensor        # int16 bit patterns of the BF16 target values


class TwoRoundTransfer:
    """Static schedule of a plan plus the two communication rounds.

    shard_receivers[k]: receiver index of shard k; op_dst_shard[o]: shard of operation o;
    op_sender[o]: sender index that owns the operation's source tensor; rank_of_sender /
    rank_of_receiver: process-group rank that plays each role (one rank may play both).
    """

    def __init__(self, shard_receivers: Sequence[int], op_dst_shard: Sequence[int], op_sender: Sequence[int],
                 rank_of_sender: Sequence[int], rank_of_receiver: Sequence[int], group=None,
                 zero_count_calls: bool = False):
        self.shard_receivers = np.asarray(shard_receivers, dtype=np.int64)
        self.op_dst_shard = np.asarray(op_dst_shard, dtype=np.int64)
        self.op_sender = np.asarray(op_sender, dtype=np.int64)
        assert self.op_dst_shard.shape == self.op_sender.shape
        self.rank_of_sender = [int(r) for r in rank_of_sender]
        self.rank_of_receiver = [int(r) for r in rank_of_receiver]
        # two routes between the same pair of ranks in one direction would share a message order
        assert len(set(self.rank_of_sender)) == len(self.rank_of_sender), "one sender role per rank"
        assert len(set(self.rank_of_receiver)) == len(self.rank_of_receiver), "one receiver role per rank"
        self.n_shards = int(self.shard_receivers.size)
        self.group = group
        # Issue the round-2 calls of a pair even when its total is zero (the paper's matched
        # zero-count calls).  Off by default: after round 1 both sides know the total, so both
        # skip the same calls and the schedule stays aligned either way.
        self.zero_count_calls = bool(zero_count_calls)
        self.check_counts = True   # sender-side consistency check before round 1 (one small host read per route)
        self.routes: Dict[Tuple[int, int], Route] = {}
        op_receiver = self.shard_receivers[self.op_dst_shard] if self.op_dst_shard.size else self.op_dst_shard
        # operations of each sender in plan order: the order of a sender's own plan and of its counts
        self.sender_ops = [np.nonzero(self.op_sender == s)[0] for s in range(len(self.rank_of_sender))]
        for s in range(len(self.rank_of_sender)):
            for r in range(len(self.rank_of_receiver)):
                ops = np.nonzero((self.op_sender == s) & (op_receiver == r))[0]
                if ops.size == 0:
                    continue                      # the plan has nothing for this pair: no calls at all
                shards = np.nonzero(self.shard_receivers == r)[0]
                slot = np.searchsorted(shards, self.op_dst_shard[ops])
                contiguous = bool(shards.size == 0 or shards[-1] - shards[0] + 1 == shards.size)
                self.routes[s, r] = Route(s, r, ops, np.searchsorted(self.sender_ops[s], ops), slot, shards,
                                          contiguous)

    # ---- helpers ---------------------------------------------------------------------------
    def routes_from(self, s: int) -> List[Route]:
        return [self.routes[k] for k in sorted(self.routes) if k[0] == s]

    def routes_to(self, r: int) -> List[Route]:
        return [self.routes[k] for k in sorted(self.routes) if k[1] == r]

    def _payload(self, route: Route, list_ptr: np.ndarray, offsets: torch.Tensor, values: torch.Tensor):
        """Entries of the receiver's lists, in list order: a view when the shards are consecutive."""
        if route.contiguous:
            a, b = int(list_ptr[route.shards[0]]), int(list_ptr[route.shards[-1] + 1])
            return offsets[a:b], values[a:b]
        parts = [(int(list_ptr[k]), int(list_ptr[k + 1])) for k in route.shards]
        return (torch.cat([offsets[a:b] for a, b in parts]), torch.cat([values[a:b] for a, b in parts]))

    def _list_ptr(self, route: Route, counts: np.ndarray) -> np.ndarray:
        per_shard = np.zeros(self.n_shards, dtype=np.uint64)
        np.add.at(per_shard, route.shards[route.op_slot], counts.astype(np.uint64))
        lp = np.zeros(self.n_shards + 1, dtype=np.uint64)
        np.cumsum(per_shard, out=lp[1:])
        return lp

    @staticmethod
    def _run(ops):
        if not ops:
            return
        for w in dist.batch_isend_irecv(ops):
            w.wait()

    # ---- the two rounds ------------------------------------------------------------------------
    def exchange(self, rank: int, sender: Optional[int], receiver: Optional[int],
                 list_ptr: Optional[np.ndarray] = None, offsets: Optional[torch.Tensor] = None,
                 values: Optional[torch.Tensor] = None, op_counts: Optional[torch.Tensor] = None,
                 device="cpu") -> Dict[int, Received]:
        """Runs both rounds on this rank.

        `sender` / `receiver`: the role indices this rank plays (None for none).  A sender passes
        its extract result: `list_ptr` (host copy, uint64[n_shards + 1]), `offsets` / `values`
        (tensors on `device`) and `op_counts` (int64 tensor on `device`: the counts of the sender's
        own operations in plan order, i.e. what dte_op_counts returns for the sender's plan).  Returns, for a receiver, one `Received` per
        sender that has a route to it (in sender order); entries are on `device`.
        """
        device = torch.device(device)
        out_routes = self.routes_from(sender) if sender is not None else []
        in_routes = self.routes_to(receiver) if receiver is not None else []
        if out_routes:
            assert list_ptr is not None and offsets is not None and values is not None and op_counts is not None
            assert op_counts.numel() == self.sender_ops[sender].size, "one count per operation of the sender"
            list_ptr = np.asarray(list_ptr, dtype=np.uint64)
        got: Dict[int, Received] = {}

        # Before anything is sent: the counts a sender is about to announce must add up to the lists
        # it holds.  After round 1 the receivers post their receives for the announced totals; a
        # sender that found a mismatch only then, and left, would keep them waiting for bytes that
        # never come - and one that left before round 1 would keep them waiting for the counts.  So
        # a sender whose lists are inconsistent stays in the schedule: it announces -1 for every
        # operation of every route (round 1 keeps its shape), sends no payload, and raises once both
        # rounds are over; a receiver that reads -1 posts no receive for that route and raises at
        # the same point.  Every rank returns or raises; none blocks.
        payloads, problems = {}, []
        for rt in out_routes:
            payloads[rt.receiver] = self._payload(rt, list_ptr, offsets, values)
            if self.check_counts:
                announced = int(op_counts[torch.as_tensor(rt.local_ops, device=op_counts.device)].sum().item())
                held = payloads[rt.receiver][0].numel()
                if announced != held:
                    problems.append(f"route {rt.sender}->{rt.receiver}: counts announce {announced} entries, "
                                    f"lists hold {held}")
        poisoned = bool(problems)

        # round 1: c_o for every operation of every pair, plan order, zeros included
        p2p, keep, count_bufs = [], [], {}
        for rt in out_routes:
            counts = op_counts[torch.as_tensor(rt.local_ops, device=op_counts.device)].to(torch.int64).contiguous()
            if poisoned:
                counts = torch.full_like(counts, -1)
            peer = self.rank_of_receiver[rt.receiver]
            if peer == rank:
                count_bufs[rt.sender] = counts
            else:
                keep.append(counts)
                p2p.append(dist.P2POp(dist.isend, counts, peer, self.group))
        for rt in in_routes:
            peer = self.rank_of_sender[rt.sender]
            if peer != rank:
                count_bufs[rt.sender] = torch.empty(rt.ops.size, dtype=torch.int64, device=device)
                p2p.append(dist.P2POp(dist.irecv, count_bufs[rt.sender], peer, self.group))
        self._run(p2p)

        # the receiver sizes its buffers (the one host read of the protocol)
        p2p, keep = [], []
        for rt in in_routes:
            counts = count_bufs[rt.sender].cpu().numpy().astype(np.int64)
            if counts.size and counts.min() < 0:
                problems.append(f"sender {rt.sender} reported inconsistent lists; nothing received from it")
                continue
            total = int(counts.sum())
            rec = Received(rt.sender, counts, self._list_ptr(rt, counts),
                           torch.empty(total, dtype=torch.int32, device=device),
                           torch.empty(total, dtype=torch.int16, device=device))
            got[rt.sender] = rec
            peer = self.rank_of_sender[rt.sender]
            if peer != rank and (total or self.zero_count_calls):
                p2p.append(dist.P2POp(dist.irecv, rec.offsets, peer, self.group))
                p2p.append(dist.P2POp(dist.irecv, rec.values, peer, self.group))

        # round 2: I_o and V_o, same order
        for rt in out_routes:
            if poisoned:
                break
            off, val = payloads[rt.receiver]
            peer = self.rank_of_receiver[rt.receiver]
            if peer == rank:
                got[rt.sender].offsets.copy_(off)
                got[rt.sender].values.copy_(val)
            elif off.numel() or self.zero_count_calls:
                off, val = off.contiguous(), val.contiguous()
                keep += [off, val]
                p2p.append(dist.P2POp(dist.isend, off, peer, self.group))
                p2p.append(dist.P2POp(dist.isend, val, peer, self.group))
        self._run(p2p)
        if problems:
            raise RuntimeError("; ".join(problems))
        return got
