"""Streaming SparseLoCo (the paper's appendix of that name): the tensor table is cut into P fragments that
take their outer steps in turn.  Each fragment is a context of its own over the same flat buffers (its
tensors keep their offsets), so a fragment's step is the ordinary sl_outer_step on a subset of the
tensors; which fragment is due after an inner step is sl_streaming_due().  Plumbing only."""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


def partition_by_layers(layers: Sequence[int], P: int) -> List[List[int]]:
    """Tensor indices of P fragments of consecutive layers, as even as the layer count allows.
    `layers[j]` = layer of tensor j, with -1 for what comes before the first layer (the embedding: goes
    into the first fragment) and any value above the last layer for what comes after it (final norm,
    unembedding: the last fragment) -- the split the paper describes for its 18-layer model."""
    real = sorted({l for l in layers if l >= 0})
    n = len(real)
    assert 1 <= P <= max(n, 1)
    bounds = [real[(p * n) // P] for p in range(P)] + [float("inf")]
    out: List[List[int]] = [[] for _ in range(P)]
    for j, l in enumerate(layers):
        if l < 0:
            out[0].append(j)
            continue
        p = max(q for q in range(P) if bounds[q] <= l) if l >= bounds[0] else 0
        out[min(p, P - 1)].append(j)
    return out


class StreamingSparseLoCo:
    """P fragment contexts over one set of flat buffers and their schedule."""

    def __init__(self, shapes, offsets, fragments: List[List[int]], *, k: int, R: int, H: int, **kw):
        self.H, self.P, self.R = H, len(fragments), R
        self.fragments = fragments
        self.ctx = [B.SparseLoCo([shapes[j] for j in f], [offsets[j] for j in f], k=k, R=R, H=H, **kw) for f in fragments]
        dev = self.ctx[0].device
        self.payloads = [[torch.zeros(c.payload_bytes(), dtype=torch.uint8, device=dev) for _ in range(R)] for c in self.ctx]

    def due(self, inner_step: int) -> int:
        return B.streaming_due(self.H, self.P, inner_step)

    def after_inner_step(self, inner_step: int, theta_sync, theta_local, e) -> Optional[int]:
        """Runs the outer step of the fragment that is due, if any; returns its number."""
        p = self.due(inner_step)
        if p < 0:
            return None
        self.ctx[p].outer_step(theta_sync, theta_local, e, self.payloads[p])
        return p

    def peak_payload_bytes(self) -> int:
        return max(c.payload_bytes() for c in self.ctx)
