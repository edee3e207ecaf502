"""sl_compress_tensor_static: the compression of one tensor for callers that cannot allocate device
memory (everything handed to an arena or caching allocator, or a section that must not take the
allocator's device-wide synchronisation).  Its scratch is a fixed 4 MiB array inside the library,
so the call needs no context and no workspace.

The check: on the same inputs it must leave exactly the bytes that the ordinary entry point,
sl_compress() on a context holding that single tensor, leaves, and that the CPU oracle computes
-- payload and error buffer bit-exact (the bar of the other GPU tests) -- on two calls in a row
that carry the error buffer over, for a blocked matrix, a flat vector with a short tail, a smaller
call after a larger one (the shared scratch keeps the previous call's contents, which must not
leak into the next), and two tensors that nearly fill the scratch.
Oversized tensors must be refused.  This file is collected last on purpose."""
import os

import pytest
import torch

from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _pair(rows, cols, k, seed):
    """Buffers for both entry points on identical seeded inputs."""
    from paper_2508_15706_b200 import binding as B
    dev = torch.device("cuda", torch.cuda.current_device())
    spec = [I.TensorSpec("t", rows, cols, 0)]
    wl = I.Workload("noalloc", spec, R=1, k=k, recipe="student_t4", seed=seed, beta=0.9)
    theta = I.theta_sync(wl, dev)
    sl = B.SparseLoCo([(rows, cols)], [0], k=k, R=1, beta=wl.beta)
    n_pay = sl.payload_bytes()
    return B, wl, theta, sl, n_pay, dev


# the last two fill most of the 4 MiB scratch (about 8,700 chunks at k = 64): a blocked matrix of 7,920
# chunks and a flat vector of 8,001 chunks with a short tail, 124 and 126 summation groups
SHAPES = [(128, 192, 64), (1, 4096 * 3 + 1234, 41), (64, 64, 123), (5632, 5760, 64), (1, 4096 * 8000 + 77, 64)]


@pytest.mark.parametrize("rows,cols,k", SHAPES)
def test_static_scratch_entry_point_matches_sl_compress(rows, cols, k):
    """Against sl_compress() on the same inputs, and both against the CPU oracle (Alg. 1, the worker's
    compression block): payload bytes and error buffer bit for bit."""
    import numpy as np
    import oracle as O
    O.set_threads(os.cpu_count() or 1)
    B, wl, theta, sl, n_pay, dev = _pair(rows, cols, k, seed=500 + k)
    e_ref = I.initial_error(wl, 0, dev, scale=0.5)
    e_new = e_ref.clone()
    e_orc = e_ref.cpu().numpy().copy()
    cfg = O.Config(k=k, R=1, beta=wl.beta)
    tab = O.Table([(rows, cols)])
    for step in range(2):  # two calls in a row, error feedback carried from the first into the second
        local = I.theta_local(wl, theta, 0, step)
        pay_ref = torch.zeros(n_pay, dtype=torch.uint8, device=dev)
        pay_new = torch.full((n_pay,), 0xAB, dtype=torch.uint8, device=dev)  # must be fully overwritten
        sl.compress(theta, local, e_ref, pay_ref)
        B.compress_tensor_static(theta, local, e_new, pay_new, rows, cols, k, wl.beta)
        torch.cuda.synchronize()
        assert torch.equal(pay_new, pay_ref), f"payload differs at step {step}"
        assert torch.equal(e_new.view(torch.int32), e_ref.view(torch.int32)), f"error buffer differs at step {step}"
        out = O.compress(cfg, tab, theta.cpu().numpy(), local.cpu().numpy(), e_orc)
        assert np.array_equal(pay_new.cpu().numpy(), out.payload), f"payload differs from the oracle at step {step}"
        assert np.array_equal(e_new.cpu().numpy().view(np.uint32), e_orc.view(np.uint32)), \
            f"error buffer differs from the oracle at step {step}"


def test_static_scratch_rejects_what_does_not_fit_and_bad_arguments():
    from paper_2508_15706_b200 import binding as B
    dev = torch.device("cuda", torch.cuda.current_device())
    assert B.static_scratch_bytes() == 4 << 20
    small = torch.zeros(4096, device=dev)
    pay = torch.zeros(4096, dtype=torch.uint8, device=dev)
    with pytest.raises(B.SlError) as ei:  # 64 Mi elements = 16384 chunks: more than the scratch holds
        B.compress_tensor_static(small, small, small.clone(), pay, 8192, 8192, 64, 0.9)
    assert ei.value.status == B.SL_ERR_TOO_LARGE
    with pytest.raises(B.SlError) as ei:
        B.compress_tensor_static(small, small, small.clone(), pay, 64, 64, 300, 0.9)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:
        B.compress_tensor_static(small, small, small.clone(), pay, 64, 64, 0, 0.9)
    assert ei.value.status == B.SL_ERR_INVALID_ARG
    with pytest.raises(B.SlError) as ei:
        B.compress_tensor_static(small, small, small.clone()[1:], pay, 1, 4095, 8, 0.9)
    assert ei.value.status == B.SL_ERR_ALIGNMENT
    torch.cuda.synchronize()
