"""The outer step with one worker per rank (Algorithm 1 as deployed: every worker compresses its own
pseudo-gradient, the payloads are all-gathered, every replica applies the same average).

    rank r:  payload_r = compress(theta, theta_r, e_r)            (Alg. 1, the worker's block; Eq. 2 lines 1-2)
    all   :  all-gather of the R payloads                         (Sec. "SparseLoCo Evaluations": ring all-gather
                                                                   of sparse payloads is what the paper counts)
    rank r:  theta = theta - alpha / D * sum_r decode(payload_r)  (Eq. 2 lines 3-4), identical on every rank

Plumbing only: the compression and the update are the library's kernels (`SparseLoCo.compress`,
`SparseLoCo.aggregate_apply`, optionally `encode_payload` / `decode_payload` for the wire), the
exchange is `torch.distributed` (NCCL on GPUs).  The gathered payloads land in this rank's own
memory and the kernels read only that: no peer pointers anywhere.

`ops` is anything with the binding's method names, so the same driver runs on CPU ranks (gloo) with
a stand-in for the kernels in the tests.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist


class PayloadExchange:
    """All-gather of one payload per rank into a [world, bytes] buffer: row r is rank r's payload.
    A rank may sit a round out (`present=False`): its row is not used and the others are told."""

    def __init__(self, payload_bytes: int, world: int, device, group=None):
        self.world, self.group = world, group
        self.gathered = torch.zeros((world, payload_bytes), dtype=torch.uint8, device=device)
        self.meta = torch.zeros((world, 2), dtype=torch.int64, device=device)  # present, bytes used

    def gather(self, own: torch.Tensor, present: bool = True, used_bytes: Optional[int] = None):
        """Returns (rows, present flags, bytes used per rank).  `own` is this rank's row (a full row long);
        `used_bytes` (default: all) is how much of it carries data, which bounds what travels."""
        n = self.gathered.shape[1]
        assert own.numel() == n and own.dtype == torch.uint8
        used = n if used_bytes is None else int(used_bytes)
        mine = torch.tensor([int(present), used if present else 0], dtype=torch.int64, device=self.meta.device)
        if self.world > 1:
            dist.all_gather(list(self.meta.unbind(0)), mine, group=self.group)
        else:
            self.meta[0].copy_(mine)
        meta = self.meta.cpu()
        flags = [bool(meta[r, 0]) for r in range(self.world)]
        sizes = [int(meta[r, 1]) for r in range(self.world)]
        width = max(sizes) if any(flags) else 0
        width = min(n, (width + 15) // 16 * 16)
        if width:
            if self.world > 1:
                rows = [self.gathered[r, :width] for r in range(self.world)]
                dist.all_gather(rows, own[:width].contiguous(), group=self.group)
            else:
                self.gathered[0, :width].copy_(own[:width])
        return [self.gathered[r] for r in range(self.world)], flags, sizes


class WorkerStep:
    """One rank of the worker-per-rank outer step.  `ops` is a context created with R = world size."""

    def __init__(self, ops, payload_bytes: int, world: int, rank: int, device, group=None, coded: bool = False,
                 coded_capacity: int = 0, expand_coded: bool = False):
        """`coded`: entropy-coded indices on the wire.  The gathered coded payloads then go straight into
        `aggregate_apply_coded` (decoding fused into the update); with `expand_coded` each is first
        expanded to the 12-bit form with `decode_payload` (what a receiver does that wants to run the
        payload validator on untrusted input) and `aggregate_apply` consumes those."""
        self.ops, self.world, self.rank, self.coded = ops, world, rank, coded
        self.expand_coded = expand_coded
        self.own = torch.zeros(payload_bytes, dtype=torch.uint8, device=device)
        if coded:
            # entropy-coded indices on the wire: about 0.68 of the plain payload at k = 64
            self.own_coded = torch.zeros(coded_capacity, dtype=torch.uint8, device=device)
            self.coded_size = torch.zeros(1, dtype=torch.int64, device=device)
            self.exchange = PayloadExchange(coded_capacity, world, device, group)
            self.plain = torch.zeros((world, payload_bytes), dtype=torch.uint8, device=device)
        else:
            self.exchange = PayloadExchange(payload_bytes, world, device, group)

    def step(self, theta_sync: torch.Tensor, theta_local: torch.Tensor, e: Optional[torch.Tensor],
             participate: bool = True) -> List[bool]:
        """Updates theta_sync (and e) in place; returns which ranks took part.  With
        `divide_by_present` set on the context the average divides by their number, else by R."""
        if participate:
            self.ops.compress(theta_sync, theta_local, e, self.own)
        if not self.coded:
            rows, flags, _ = self.exchange.gather(self.own, participate)
            payloads = [rows[r] if flags[r] else None for r in range(self.world)]
        else:
            used = 0
            if participate:
                self.ops.encode_payload(self.own, self.own_coded, self.coded_size)
                used = int(self.coded_size.item())
            rows, flags, sizes = self.exchange.gather(self.own_coded, participate, used)
            if not self.expand_coded:
                self.ops.aggregate_apply_coded([rows[r] if flags[r] else None for r in range(self.world)], theta_sync,
                                               sizes)
                return flags
            payloads = []
            for r in range(self.world):
                if not flags[r]:
                    payloads.append(None)
                    continue
                self.ops.decode_payload(rows[r], self.plain[r], coded_bytes=sizes[r])
                payloads.append(self.plain[r])
        self.ops.aggregate_apply(payloads, theta_sync)
        return flags
