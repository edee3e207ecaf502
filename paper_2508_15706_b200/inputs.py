"""Seeded synthetic inputs for the SparseLoCo outer step.

This module is the only code shared by the CUDA path's tests/bench and the CPU
oracle's tests.  It holds tensor-shape lists and random-number recipes only:
none of the method's arithmetic (no pseudo-gradient, no Top-k, no quantiser)
lives here.  Every array it returns is a plain fp32 torch tensor on the device
the caller names, so the same bytes can be handed to both sides.

Shapes: Llama-style decoder stacks (untied embedding and output head, q/k/v/o
projections, SwiGLU gate/up/down, two norm vectors per layer and a final norm;
the MoE variant adds a router and per-expert gate/up/down).  They stand in for
the pseudo-gradients of the models the paper trains on DCLM (Experiments
section; model tables in the appendix), which cannot be reproduced without the
dataset and trained weights.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import torch


@dataclass(frozen=True)
class TensorSpec:
    """One parameter tensor of a model: `rows x cols` fp32, 1-D when rows == 1."""
    name: str
    rows: int
    cols: int
    layer: int  # -1 for embed / lm_head / final norm
    expert: int = -1  # >= 0 for MoE expert matrices

    @property
    def numel(self) -> int:
        return self.rows * self.cols


def dense_transformer(d_model: int, n_layers: int, ffn: int, vocab: int,
                      kv_dim: Optional[int] = None) -> List[TensorSpec]:
    """Tensor list of a dense decoder; `kv_dim` < d_model gives grouped-query k/v projections."""
    kv = d_model if kv_dim is None else kv_dim
    t: List[TensorSpec] = [TensorSpec("embed", vocab, d_model, -1)]
    for l in range(n_layers):
        for nm in ("q", "k", "v", "o"):
            t.append(TensorSpec(f"l{l}.{nm}", kv if nm in ("k", "v") else d_model, d_model, l))
        t.append(TensorSpec(f"l{l}.gate", ffn, d_model, l))
        t.append(TensorSpec(f"l{l}.up", ffn, d_model, l))
        t.append(TensorSpec(f"l{l}.down", d_model, ffn, l))
        t.append(TensorSpec(f"l{l}.norm1", 1, d_model, l))
        t.append(TensorSpec(f"l{l}.norm2", 1, d_model, l))
    t.append(TensorSpec("final_norm", 1, d_model, -1))
    t.append(TensorSpec("lm_head", vocab, d_model, -1))
    return t


def moe_transformer(d_model: int, n_layers: int, n_experts: int, ffn: int, vocab: int) -> List[TensorSpec]:
    t: List[TensorSpec] = [TensorSpec("embed", vocab, d_model, -1)]
    for l in range(n_layers):
        for nm in ("q", "k", "v", "o"):
            t.append(TensorSpec(f"l{l}.{nm}", d_model, d_model, l))
        t.append(TensorSpec(f"l{l}.router", n_experts, d_model, l))
        for x in range(n_experts):
            t.append(TensorSpec(f"l{l}.x{x}.gate", ffn, d_model, l, x))
            t.append(TensorSpec(f"l{l}.x{x}.up", ffn, d_model, l, x))
            t.append(TensorSpec(f"l{l}.x{x}.down", d_model, ffn, l, x))
        t.append(TensorSpec(f"l{l}.norm1", 1, d_model, l))
        t.append(TensorSpec(f"l{l}.norm2", 1, d_model, l))
    t.append(TensorSpec("final_norm", 1, d_model, -1))
    t.append(TensorSpec("lm_head", vocab, d_model, -1))
    return t


@dataclass(frozen=True)
class Workload:
    """A named benchmark/parity configuration (shapes + hyper-parameters + recipe)."""
    name: str
    tensors: Sequence[TensorSpec]
    R: int
    k: int
    H: int = 15
    beta: float = 0.95
    outer_lr: float = 1.0
    steps: int = 1
    recipe: str = "normal"  # normal | outlier_ties | student_t4 | moe_zero
    seed: int = 0
    k_sweep: Sequence[int] = field(default_factory=tuple)

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)


def workload(name: str) -> Workload:
    """The five configurations of the benchmark contract, by short name."""
    if name == "c1_single_1024":
        return Workload(name, [TensorSpec("w", 1024, 1024, 0)], R=2, k=64, H=1,
                        recipe="outlier_ties", seed=0)
    if name == "c2_dense_d768":
        return Workload(name, dense_transformer(768, 12, 3072, 32000), R=8, k=64, H=15,
                        steps=3, recipe="normal", seed=2)
    if name == "c3_dense_d1280":
        return Workload(name, dense_transformer(1280, 24, 5120, 32000), R=8, k=82, H=15,
                        steps=2, recipe="student_t4", seed=3, k_sweep=(41, 82, 123))
    if name == "c4_moe_d1024":
        return Workload(name, moe_transformer(1024, 12, 8, 2048, 32000), R=8, k=64, H=15,
                        steps=2, recipe="moe_zero", seed=4)
    if name == "c5_dense_d2048":
        return Workload(name, dense_transformer(2048, 24, 8192, 32000), R=16, k=64, H=30,
                        outer_lr=0.8, recipe="normal", seed=5)
    if name == "c5_l12":  # half the depth of c5_dense_d2048: 16 distinct theta_local AND 16 e buffers fit one GPU
        return Workload(name, dense_transformer(2048, 12, 8192, 32000), R=16, k=64, H=30,
                        outer_lr=0.8, recipe="normal", seed=5)
    if name == "c5_layer0":  # one decoder layer of c5_dense_d2048: small enough to profile
        full = dense_transformer(2048, 24, 8192, 32000)
        return Workload(name, [t for t in full if t.layer == 0], R=16, k=64, H=30,
                        outer_lr=0.8, recipe="normal", seed=5)
    raise KeyError(name)


WORKLOADS = ("c1_single_1024", "c2_dense_d768", "c3_dense_d1280", "c4_moe_d1024", "c5_dense_d2048")


def offsets(tensors: Sequence[TensorSpec], align: int = 4) -> List[int]:
    """Element offset of every tensor in a flat buffer, each rounded up to `align` elements."""
    out, pos = [], 0
    for t in tensors:
        pos = (pos + align - 1) // align * align
        out.append(pos)
        pos += t.numel
    return out


def flat_numel(tensors: Sequence[TensorSpec], align: int = 4) -> int:
    off = offsets(tensors, align)
    return off[-1] + tensors[-1].numel if tensors else 0


def _gen(device, *parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for p in parts:
        s = ((s ^ (int(p) + 0x632BE59BD9B4E019)) * 0xD1342543DE82EF95) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(s)
    return g


def _student_t(n: int, df: int, g: torch.Generator, device) -> torch.Tensor:
    z = torch.randn(n, generator=g, device=device)
    chi = torch.zeros(n, device=device)
    for _ in range(df):
        chi += torch.randn(n, generator=g, device=device) ** 2
    return z / torch.sqrt(chi / df)


def layer_sigma(wl: Workload, layer: int) -> float:
    """Per-layer pseudo-gradient scale, log-uniform in [1e-4, 1e-2] (seeded)."""
    g = _gen("cpu", wl.seed, 77, layer + 1)
    u = torch.rand(1, generator=g).item()
    return 10.0 ** (-4.0 + 2.0 * u)


def theta_sync(wl: Workload, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Synchronised parameters: N(0, 0.02) in every tensor, flat fp32 buffer."""
    n = flat_numel(wl.tensors)
    buf = out if out is not None else torch.zeros(n, dtype=torch.float32, device=device)
    for ti, (t, off) in enumerate(zip(wl.tensors, offsets(wl.tensors))):
        g = _gen(device, wl.seed, 1, ti)
        buf[off:off + t.numel].normal_(0.0, 0.02, generator=g)
    if wl.recipe == "outlier_ties":  # tied positions: theta_sync is exactly zero there
        t = wl.tensors[0]
        ts2 = buf[:t.numel].view(t.rows, t.cols)
        for tile, entry in tie_plan(wl).items():
            tr, tc = divmod(tile, t.cols // 64)
            for key_pos in ("pos", "low_pos"):
                if key_pos in entry:
                    pos = entry[key_pos].to(buf.device)
                    ts2[tr * 64 + pos // 64, tc * 64 + pos % 64] = 0.0
    return buf


def zero_experts(wl: Workload, worker: int, step: int, layer: int, n_experts: int = 8) -> List[int]:
    """MoE recipe: the experts (30 %, at least 2) that worker `worker` did not route to."""
    g = _gen("cpu", wl.seed, 55, worker, step, layer)
    n_zero = max(2, int(round(0.3 * n_experts)))
    return sorted(torch.randperm(n_experts, generator=g)[:n_zero].tolist())


def delta_tensor(wl: Workload, ti: int, worker: int, step: int, device="cpu") -> torch.Tensor:
    """The drift one worker's inner loop adds to tensor `ti` (flat, fp32): theta_local is
    theta_sync minus this.  Distribution follows `wl.recipe`."""
    t = wl.tensors[ti]
    n = t.numel
    g = _gen(device, wl.seed, 1000 + worker, step, ti)
    if wl.recipe == "outlier_ties":
        d = torch.randn(n, generator=g, device=device) * 1e-3
        mask = torch.rand(n, generator=g, device=device) < 0.05
        heavy = _student_t(n, 3, g, device) * 1e-3
        d = torch.where(mask, heavy, d)
        return d
    sig = layer_sigma(wl, t.layer)
    if wl.recipe == "normal":
        return torch.randn(n, generator=g, device=device) * sig
    if wl.recipe == "student_t4":
        return _student_t(n, 4, g, device) * sig
    if wl.recipe == "moe_zero":
        if t.expert >= 0 and t.expert in zero_experts(wl, worker, step, t.layer):
            return torch.zeros(n, device=device)
        return torch.randn(n, generator=g, device=device) * sig
    raise ValueError(wl.recipe)


def tie_plan(wl: Workload) -> Dict[int, dict]:
    """`outlier_ties` recipe: which 64x64 tiles of the single 1024x1024 tensor carry exact
    ties, and where.  Returns {tile_id: {"pos": LongTensor of in-tile positions (row-major in
    the tile), "mag": float, "low_pos": optional positions of a second, small tie group}}."""
    g = _gen("cpu", wl.seed, 99)
    plan: Dict[int, dict] = {}
    tiles = torch.randperm(256, generator=g)[:3].tolist()
    for j, tile in enumerate(tiles):
        perm = torch.randperm(4096, generator=g)
        entry = {"pos": perm[:100].sort().values, "mag": 2.0 ** -6}
        if j == 2:  # ties below the cut as well: must be ignored by the selection
            entry["low_pos"] = perm[100:220].sort().values
            entry["low_mag"] = 2.0 ** -20
        plan[tile] = entry
    return plan


def theta_local(wl: Workload, theta_s: torch.Tensor, worker: int, step: int,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One worker's parameters after its inner loop: theta_sync minus the seeded drift.
    `outlier_ties` additionally plants exact ties (see `tie_plan`): theta_sync is zero at the
    tied positions and theta_local is +-mag there, so the difference is exactly -+mag."""
    device = theta_s.device
    buf = out if out is not None else torch.empty_like(theta_s)
    offs = offsets(wl.tensors)
    for ti, (t, off) in enumerate(zip(wl.tensors, offs)):
        d = delta_tensor(wl, ti, worker, step, device)
        torch.sub(theta_s[off:off + t.numel], d, out=buf[off:off + t.numel])
        del d
    if wl.recipe == "outlier_ties":
        t = wl.tensors[0]
        tl2 = buf[:t.numel].view(t.rows, t.cols)
        for tile, entry in tie_plan(wl).items():
            tr, tc = divmod(tile, t.cols // 64)
            sgen = _gen("cpu", wl.seed, 98, worker, tile)
            for key_pos, key_mag in (("pos", "mag"), ("low_pos", "low_mag")):
                if key_pos not in entry:
                    continue
                pos = entry[key_pos].to(device)
                rr = tr * 64 + pos // 64
                cc = tc * 64 + pos % 64
                sign = (torch.randint(0, 2, (pos.numel(),), generator=sgen) * 2 - 1).to(
                    device=device, dtype=torch.float32)
                tl2[rr, cc] = sign * entry[key_mag]
    return buf


def initial_error(wl: Workload, worker: int, device="cpu", scale: float = 0.0,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Error-feedback buffer before the first step: zeros (Algorithm 1's e^(0) = 0) or, with
    `scale` > 0, seeded noise of `scale` x the layer's drift scale (used by the bench so
    that workers sharing a theta_local buffer still differ)."""
    n = flat_numel(wl.tensors)
    buf = out if out is not None else torch.zeros(n, dtype=torch.float32, device=device)
    if scale == 0.0:
        buf.zero_()
        return buf
    for ti, (t, off) in enumerate(zip(wl.tensors, offsets(wl.tensors))):
        g = _gen(device, wl.seed, 2000 + worker, ti)
        sig = layer_sigma(wl, t.layer) if wl.recipe != "outlier_ties" else 1e-3
        buf[off:off + t.numel].normal_(0.0, scale * sig, generator=g)
    return buf
