"""Helpers for the GPU-vs-oracle parity tests (not a test module).

The CUDA path runs on the whole workload; the oracle is run tensor by tensor on copies taken
before the step (every stage of the method is per tensor, so a tensor can be checked alone).
Bars: payload bytes (indices, codes, tables) and error buffers bit-exact; theta_sync within
1e-6 x RMS(tensor) of the oracle's fp64 evaluation.
"""
from __future__ import annotations

import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

import oracle as O
from paper_2508_15706_b200 import inputs as I

THETA_TOL_REL_RMS = 1e-6


def oracle_threads() -> int:
    n = os.cpu_count() or 1
    O.set_threads(n)
    return n


GUARD_BYTES = 4096   # on either side of every buffer the kernels write
CANARY = 0xC5


class Guarded:
    """A device buffer with a band of known bytes before and after it.  The kernels get the middle;
    `intact()` tells whether anything wrote outside it (the stand-in for a memory checker)."""

    def __init__(self, numel: int, dtype, device, extra_bytes: int = 0):
        item = torch.empty((), dtype=dtype).element_size()
        self.n_bytes = numel * item
        total = GUARD_BYTES + (self.n_bytes + extra_bytes + 255) // 256 * 256 + GUARD_BYTES
        self.raw = torch.full((total,), CANARY, dtype=torch.uint8, device=device)
        self.view = self.raw[GUARD_BYTES:GUARD_BYTES + self.n_bytes].view(dtype)
        self.tail_from = GUARD_BYTES + self.n_bytes + extra_bytes

    def intact(self) -> bool:
        return bool((self.raw[:GUARD_BYTES] == CANARY).all()) and bool((self.raw[self.tail_from:] == CANARY).all())


class DeviceCase:
    """Device-resident buffers of one workload: theta_sync, D distinct theta_local buffers
    (worker r reads buffer r % D, through a view shifted by (r // D) * alias_shift elements, as
    bench.py arranges them), R error buffers, R payloads, the workspace.  Everything the kernels
    write sits between guard bands, which check() and step() verify."""

    def __init__(self, wl: I.Workload, k: Optional[int] = None, distinct_local: Optional[int] = None,
                 e_scale: float = 0.0, device=None, alias_shift: int = 0, quant_bits: int = 2):
        from paper_2508_15706_b200.binding import SparseLoCo
        self.wl = wl
        self.k = wl.k if k is None else k
        self.dev = device or torch.device("cuda", torch.cuda.current_device())
        self.offs = I.offsets(wl.tensors)
        self.shapes = [(t.rows, t.cols) for t in wl.tensors]
        self.D = wl.R if distinct_local is None else distinct_local
        self.alias_shift = alias_shift if self.D < wl.R else 0
        self.quant_bits = quant_bits
        self.sl = SparseLoCo(self.shapes, self.offs, k=self.k, R=wl.R, H=wl.H, beta=wl.beta,
                             outer_lr=wl.outer_lr, alloc_workspace=False, quant_bits=quant_bits)
        flat = I.flat_numel(wl.tensors)
        self.flat = flat
        self.guarded: List[Guarded] = []

        def guarded(numel, dtype):
            g = Guarded(numel, dtype, self.dev)
            self.guarded.append(g)
            return g.view

        self.theta = guarded(flat, torch.float32)
        self.theta.zero_()
        I.theta_sync(wl, self.dev, out=self.theta)
        extra = self.alias_shift * ((wl.R + self.D - 1) // self.D - 1)
        self.local = [torch.empty(flat + extra, dtype=torch.float32, device=self.dev) for _ in range(self.D)]
        if extra:
            for d, buf in enumerate(self.local):
                g = torch.Generator(device=self.dev).manual_seed(77_000 + d)
                buf[flat:].normal_(0.0, 0.02, generator=g)
        self.e = []
        for r in range(wl.R):
            buf = guarded(flat, torch.float32)
            buf.zero_()
            I.initial_error(wl, r, self.dev, scale=e_scale, out=buf)
            self.e.append(buf)
        self.payloads = []
        for _ in range(wl.R):
            buf = guarded(self.sl.payload_bytes(), torch.uint8)
            buf.zero_()
            self.payloads.append(buf)
        self.ws = guarded(self.sl.workspace_bytes(), torch.uint8)
        self.sl.set_workspace(self.ws)
        self.cfg = O.Config(k=self.k, R=wl.R, H=wl.H, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=quant_bits)
        # payload geometry, from the oracle's definitions
        self.rec_off, self.n_chunks = [], []
        stride = O.record_stride_q(self.k, quant_bits)
        self.hdr = O.header_bytes(quant_bits)
        pos = self.hdr * len(self.shapes)
        for j, sh in enumerate(self.shapes):
            nc = O.num_chunks(self.cfg, O.Table([sh]), 0)
            self.rec_off.append(pos)
            self.n_chunks.append(nc)
            pos += nc * stride
        self.payload_bytes = pos
        self.stride = stride

    def fill_local(self, step: int) -> None:
        for d in range(self.D):
            I.theta_local(self.wl, self.theta, d, step, out=self.local[d])

    def local_of(self, r: int) -> torch.Tensor:
        o = (r // self.D) * self.alias_shift
        return self.local[r % self.D][o:o + self.flat]

    def guards_intact(self) -> bool:
        return all(g.intact() for g in self.guarded)

    def snapshot(self, tensor_ids: Sequence[int], spare: Optional[torch.Tensor] = None) -> Dict[int, dict]:
        """CPU copies of theta_sync / theta_local / e slices of the given tensors (pre-step)."""
        snap = {}
        for j in tensor_ids:  # parameters first: `spare` may be one of the theta_local buffers
            t, off = self.wl.tensors[j], self.offs[j]
            sl = slice(off, off + t.numel)
            snap[j] = {
                "theta": self.theta[sl].cpu().numpy().copy(),
                "local": [self.local_of(r)[sl].cpu().numpy().copy() for r in range(self.wl.R)],
            }
        e_cpu = self.error_slices(tensor_ids, spare=spare)
        for j in tensor_ids:
            snap[j]["e"] = [e_cpu[r][j] for r in range(self.wl.R)]
        return snap

    def step(self) -> None:
        self.sl.outer_step(self.theta, [self.local_of(r) for r in range(self.wl.R)], self.e, self.payloads)
        assert self.sl.device_status() == 0, "a kernel recorded a device-side error"
        assert self.guards_intact(), "a kernel wrote outside one of its output buffers"

    def tensor_payload(self, r: int, j: int) -> np.ndarray:
        p = self.payloads[r]
        hdr = p[self.hdr * j:self.hdr * (j + 1)].cpu().numpy()
        recs = p[self.rec_off[j]:self.rec_off[j] + self.n_chunks[j] * self.stride].cpu().numpy()
        return np.concatenate([hdr, recs])

    def true_error(self) -> List[torch.Tensor]:
        """The error buffers as the method defines them.  With the deferred subtraction on, the values
        still waiting in the workspace are written into copies (they keep waiting for the next step)."""
        if not self.sl.ef_pending():
            return self.e
        copies = [x.clone() for x in self.e]
        self.sl.ef_flush(copies, keep_pending=True)
        return copies

    def error_slices(self, tensor_ids: Sequence[int], spare: Optional[torch.Tensor] = None) -> List[Dict[int, np.ndarray]]:
        """CPU copies of the true error of the given tensors, per worker.  Large cases materialise
        one worker at a time into a single spare buffer (`spare`, at least a flat buffer long, or a
        fresh allocation)."""
        def cut(buf):
            return {j: buf[self.offs[j]:self.offs[j] + self.wl.tensors[j].numel].cpu().numpy().copy()
                    for j in tensor_ids}
        if not self.sl.ef_pending():
            return [cut(x) for x in self.e]
        out = []
        own = spare is None
        spare = torch.empty_like(self.e[0]) if own else spare[:self.flat]
        for r in range(self.wl.R):
            spare.copy_(self.e[r])
            self.sl.ef_flush([spare if q == r else None for q in range(self.wl.R)], keep_pending=True)
            torch.cuda.synchronize()
            out.append(cut(spare))
        if own:
            del spare
        return out

    def check(self, snap: Dict[int, dict], ef_enabled: bool = True, present: Optional[List[bool]] = None,
              spare: Optional[torch.Tensor] = None) -> dict:
        """Run the oracle on the snapshot tensors and compare with the device state after step()."""
        torch.cuda.synchronize()
        e_cpu = self.error_slices(list(snap.keys()), spare=spare)
        R = self.wl.R
        worst = 0.0
        report = {"tensors": 0, "payload_bytes": 0, "theta_max_err_over_rms": 0.0}
        cfg = O.Config(k=self.k, R=R, H=self.wl.H, beta=self.wl.beta, outer_lr=self.wl.outer_lr,
                       ef_enabled=int(ef_enabled), quant_bits=self.quant_bits)
        for j, s in snap.items():
            t, off = self.wl.tensors[j], self.offs[j]
            tab = O.Table([(t.rows, t.cols)])
            th = s["theta"].copy()
            pays = []
            for r in range(R):
                e_o = s["e"][r].copy()
                out = O.compress(cfg, tab, s["theta"], s["local"][r], e_o)
                got = self.tensor_payload(r, j)
                if not np.array_equal(got, out.payload):
                    bad = np.nonzero(got != out.payload)[0]
                    raise AssertionError(
                        f"payload mismatch: tensor {j} ({t.name}) worker {r}: {bad.size} bytes differ, first at "
                        f"{bad[0]} (record {(bad[0] - 16) // self.stride if bad[0] >= 16 else 'header'})")
                e_g = e_cpu[r][j]
                if not np.array_equal(e_g.view(np.uint32), e_o.view(np.uint32)):
                    bad = np.nonzero(e_g.view(np.uint32) != e_o.view(np.uint32))[0]
                    raise AssertionError(f"error buffer mismatch: tensor {j} ({t.name}) worker {r}: "
                                         f"{bad.size} elements, first {bad[0]}: {e_g[bad[0]]} vs {e_o[bad[0]]}")
                pays.append(out.payload if (present is None or present[r]) else None)
                report["payload_bytes"] += out.payload.size
            O.aggregate_apply(cfg, tab, pays, th)
            th_g = self.theta[off:off + t.numel].cpu().numpy()
            rms = float(np.sqrt(np.mean(th.astype(np.float64) ** 2)))
            err = float(np.max(np.abs(th_g.astype(np.float64) - th.astype(np.float64))))
            assert err <= THETA_TOL_REL_RMS * rms, f"theta mismatch: tensor {j} ({t.name}): {err} vs rms {rms}"
            worst = max(worst, err / rms if rms > 0 else 0.0)
            report["tensors"] += 1
        report["theta_max_err_over_rms"] = worst
        return report


def sample_tensor_ids(wl: I.Workload, want_names: Sequence[str]) -> List[int]:
    names = [t.name for t in wl.tensors]
    return [names.index(n) for n in want_names if n in names]
