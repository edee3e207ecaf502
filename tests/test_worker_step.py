"""The worker-per-rank outer step (Alg. 1 as deployed; the exchange the paper counts is an all-gather of
the sparse payloads).  On CPU: gloo ranks run the driver with the oracle standing in for the kernels and
the result must equal the oracle's single-process outer step over the same workers -- this pins the
gather order (row r = rank r), the sizes on the wire, the entropy-coded variant and the absent-rank
policy (a NULL payload; divisor R or the number present).  On a GPU: sl_aggregate_apply is fed the
payloads as one gathered [R, bytes] buffer, the layout the all-gather leaves."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


_WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
mode, world = sys.argv[2], int(os.environ["WORLD_SIZE"])
rank = int(os.environ["RANK"])
import numpy as np, torch, torch.distributed as dist
import oracle as O
from paper_2508_15706_b200 import inputs as I
from paper_2508_15706_b200.worker_step import WorkerStep

dist.init_process_group("gloo")
tensors = [I.TensorSpec("w", 128, 128, 0), I.TensorSpec("v", 1, 5000, 0), I.TensorSpec("n", 1, 300, 1)]
wl = I.Workload("ranks", tensors, R=world, k=32, recipe="normal", seed=17, outer_lr=0.7)
by_present = mode.endswith("present")
cfg = O.Config(k=wl.k, R=world, beta=wl.beta, outer_lr=wl.outer_lr, divide_by_present=int(by_present))
tab = O.Table([(t.rows, t.cols) for t in tensors], I.offsets(tensors))


class OracleOps:  # the binding's method names over the CPU oracle (the kernels' stand-in on CPU ranks)
    def compress(self, theta, local, e, payload):
        out = O.compress(cfg, tab, theta.numpy(), local.numpy(), e.numpy())
        payload.copy_(torch.from_numpy(out.payload))
    def aggregate_apply(self, payloads, theta):
        O.aggregate_apply(cfg, tab, [None if p is None else p.numpy().copy() for p in payloads], theta.numpy())
    def encode_payload(self, payload, coded, size):
        c = O.ixc_encode_payload(cfg, tab, payload.numpy())
        coded.zero_()
        coded[:c.size] = torch.from_numpy(c)
        size[0] = c.size
    def decode_payload(self, coded, payload, coded_bytes=0):
        payload.copy_(torch.from_numpy(O.ixc_decode_payload(cfg, tab, coded[:coded_bytes].numpy().copy())))
    def aggregate_apply_coded(self, coded, theta, sizes):
        plain = [None if c is None else O.ixc_decode_payload(cfg, tab, c[:n].numpy().copy()) for c, n in zip(coded, sizes)]
        O.aggregate_apply(cfg, tab, plain, theta.numpy())


theta = I.theta_sync(wl, "cpu")
local = I.theta_local(wl, theta, rank, 0)
e = I.initial_error(wl, rank, "cpu", scale=0.5)
nbytes = O.payload_bytes(cfg, tab)
coded = mode.startswith("coded")
expand = mode == "coded_expand"
ws = WorkerStep(OracleOps(), nbytes, world, rank, "cpu", coded=coded, coded_capacity=2 * nbytes, expand_coded=expand)
sits_out = mode.startswith("absent") and rank == world - 1
flags = ws.step(theta, local, e, participate=not sits_out)

# what one process computes for the same workers
theta_ref = I.theta_sync(wl, "cpu").numpy()
pays = []
for r in range(world):
    e_r = I.initial_error(wl, r, "cpu", scale=0.5).numpy()
    out = O.compress(cfg, tab, theta_ref, I.theta_local(wl, torch.from_numpy(theta_ref), r, 0).numpy(), e_r)
    absent = mode.startswith("absent") and r == world - 1
    pays.append(None if absent else out.payload)
    if r == rank and not absent:
        assert np.array_equal(e.numpy().view(np.uint32), e_r.view(np.uint32))
        assert np.array_equal(ws.own.numpy(), out.payload)
O.aggregate_apply(cfg, tab, pays, theta_ref)
same = bool(np.array_equal(theta.numpy().view(np.uint32), theta_ref.view(np.uint32)))
def row(r):
    if not coded:
        return ws.exchange.gathered[r].numpy()
    if expand:
        return ws.plain[r].numpy()
    n = int(ws.exchange.meta[r, 1])   # the gathered coded row, expanded here
    return O.ixc_decode_payload(cfg, tab, ws.exchange.gathered[r][:n].numpy().copy())
rows_ok = all(p is None or np.array_equal(row(r), p) for r, p in enumerate(pays))
wire = int(ws.exchange.meta[:, 1].max())
dist.barrier()
print(json.dumps({"rank": rank, "same": same, "rows_ok": rows_ok, "flags": flags, "wire": wire, "plain": nbytes}))
dist.destroy_process_group()
"""


@pytest.mark.parametrize("mode,world", [("plain", 2), ("plain", 3), ("coded", 2), ("coded_expand", 2), ("absent_R", 3), ("absent_present", 3)])
def test_worker_per_rank_step_equals_one_process_step(tmp_path, mode, world):
    port = _free_port()
    script = tmp_path / "w.py"
    script.write_text(_WORKER)
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT, mode], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    for rank, (so, _) in enumerate(outs):
        got = json.loads(so.strip().splitlines()[-1])
        assert got["rank"] == rank and got["same"] and got["rows_ok"], got
        want_flags = [not (mode.startswith("absent") and r == world - 1) for r in range(world)]
        assert got["flags"] == want_flags
        if mode.startswith("coded"):
            assert got["wire"] < got["plain"]      # fewer bytes travel than the 12-bit form has
        else:
            assert got["wire"] == got["plain"]


@pytest.mark.gpu
def test_aggregate_apply_from_a_gathered_buffer():
    """sl_aggregate_apply reading its R payloads as rows of one [R, bytes] buffer (what the all-gather
    leaves in local memory), one row absent: theta equals the step with separately allocated payloads."""
    import torch
    from paper_2508_15706_b200 import inputs as I
    from paper_2508_15706_b200.binding import SparseLoCo
    from paper_2508_15706_b200.worker_step import WorkerStep
    dev = torch.device("cuda", torch.cuda.current_device())
    tensors = [I.TensorSpec("w", 256, 192, 0), I.TensorSpec("v", 1, 9000, 0)]
    R = 4
    wl = I.Workload("gathered", tensors, R=R, k=64, recipe="student_t4", seed=23, outer_lr=0.9)
    shapes, offs = [(t.rows, t.cols) for t in tensors], I.offsets(tensors)
    sl = SparseLoCo(shapes, offs, k=wl.k, R=R, beta=wl.beta, outer_lr=wl.outer_lr, divide_by_present=True)
    theta = I.theta_sync(wl, dev)
    theta2 = theta.clone()
    nbytes = sl.payload_bytes()
    assert nbytes % 16 == 0                       # every row of the gathered buffer is 16-byte aligned
    gathered = torch.zeros((R, nbytes), dtype=torch.uint8, device=dev)
    separate = []
    for r in range(R):
        local = I.theta_local(wl, theta, r, 0)
        e = I.initial_error(wl, r, dev, scale=0.5)
        p = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
        sl.compress(theta, local, e, p)
        separate.append(p)
        gathered[r].copy_(p)
    present = [True, True, False, True]
    sl.aggregate_apply([separate[r] if present[r] else None for r in range(R)], theta)
    sl.aggregate_apply([gathered[r] if present[r] else None for r in range(R)], theta2)
    torch.cuda.synchronize()
    assert torch.equal(theta.view(torch.int32), theta2.view(torch.int32))
    # and the driver itself with a world of one rank (no process group): compress, "gather", apply
    sl1 = SparseLoCo(shapes, offs, k=wl.k, R=1, beta=wl.beta, outer_lr=wl.outer_lr)
    ws = WorkerStep(sl1, sl1.payload_bytes(), 1, 0, dev)
    th_a, th_b = I.theta_sync(wl, dev), I.theta_sync(wl, dev)
    local = I.theta_local(wl, th_a, 0, 0)
    e_a, e_b = I.initial_error(wl, 0, dev, scale=0.5), I.initial_error(wl, 0, dev, scale=0.5)
    assert ws.step(th_a, local, e_a) == [True]
    pay = torch.zeros(sl1.payload_bytes(), dtype=torch.uint8, device=dev)
    sl1.outer_step(th_b, [local], [e_b], [pay])
    torch.cuda.synchronize()
    assert torch.equal(th_a.view(torch.int32), th_b.view(torch.int32)) and torch.equal(e_a, e_b) and torch.equal(ws.own, pay)
