"""GPU parity of the dense baseline (DiLoCo's outer step, Eq. 1) against the oracle: theta and the
momentum within 1e-6 x RMS of the fp64 evaluation over several steps, untouched gaps between
tensors, and -- with beta = 0, alpha = 1 -- plain parameter averaging."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu

SHAPES = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("flat", 1, 5000, 0), I.TensorSpec("tiny", 1, 41, 1),
          I.TensorSpec("b", 64, 128, 2), I.TensorSpec("mid", 1, 4096 + 2051, 3)]


@pytest.mark.parametrize("R", [1, 5, 16])
def test_diloco_step_matches_oracle(R):
    from paper_2508_15706_b200.binding import SparseLoCo
    dev = torch.device("cuda", torch.cuda.current_device())
    wl = I.Workload("dense", SHAPES, R=R, k=8, recipe="normal", seed=800 + R, outer_lr=0.7)
    offs = I.offsets(SHAPES)           # 41 elements leave a gap of 3 before the next tensor
    shapes = [(t.rows, t.cols) for t in SHAPES]
    sl = SparseLoCo(shapes, offs, k=8, R=R, outer_lr=0.7, alloc_workspace=False)
    tab = O.Table(shapes, offs)
    theta = I.theta_sync(wl, dev)
    mom = torch.zeros_like(theta)
    gap = slice(offs[2] + 41, offs[3])
    theta[gap] = 123.0
    mom[gap] = -7.0
    th_o, m_o = theta.cpu().numpy().copy(), mom.cpu().numpy().copy()
    for step in range(3):
        local = [I.theta_local(wl, theta, r, step) for r in range(R)]
        loc_o = [(th_o - (theta - l).cpu().numpy()).astype(np.float32) for l in local]  # same drifts around the oracle's theta
        # feed both sides identical inputs: the device copy of the oracle's parameters
        theta.copy_(torch.from_numpy(th_o))
        mom.copy_(torch.from_numpy(m_o))
        local = [torch.from_numpy(x).to(dev) for x in loc_o]
        sl.diloco_step(theta, local, mom, 0.9)
        torch.cuda.synchronize()
        O.diloco_step(tab, th_o, loc_o, m_o, 0.9, 0.7)
        for got, want in ((theta, th_o), (mom, m_o)):
            g = got.cpu().numpy().astype(np.float64)
            for t, off in zip(SHAPES, offs):
                w = want[off:off + t.numel].astype(np.float64)
                rms = float(np.sqrt(np.mean(w ** 2))) + 1e-30
                assert np.max(np.abs(g[off:off + t.numel] - w)) <= 1e-6 * rms, (t.name, step)
        assert torch.all(theta[gap] == 123.0) and torch.all(mom[gap] == -7.0)
    # beta = 0, alpha = 1: parameter averaging
    sl2 = SparseLoCo(shapes, offs, k=8, R=R, outer_lr=1.0, alloc_workspace=False)
    mom.zero_()
    th_before = theta.clone()
    sl2.diloco_step(theta, local, mom, 0.0)
    torch.cuda.synchronize()
    avg = torch.stack([l.double() for l in local]).mean(0)
    for t, off in zip(SHAPES, offs):
        assert torch.allclose(theta[off:off + t.numel].double(), avg[off:off + t.numel], rtol=0, atol=2e-7)
    assert torch.all(theta[gap] == th_before[gap])
