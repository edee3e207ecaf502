"""Streaming SparseLoCo (the paper's appendix of that name): the fragment schedule on the CPU (no device
work), and on a GPU two full rounds of fragment-wise outer steps against the oracle taking the same
fragment steps."""
import numpy as np
import pytest


def test_schedule_every_fragment_once_per_interval_in_turn():
    from paper_2508_15706_b200 import binding as B
    # the paper's setting: H = 15 for the full model, three fragments, one synchronisation every 5 steps
    seq = [(t, B.streaming_due(15, 3, t)) for t in range(1, 46)]
    due = [(t, p) for t, p in seq if p >= 0]
    assert due == [(5, 0), (10, 1), (15, 2), (20, 0), (25, 1), (30, 2), (35, 0), (40, 1), (45, 2)]
    for H, P in ((15, 3), (30, 4), (7, 7), (8, 3), (50, 1)):
        hits = [B.streaming_due(H, P, t) for t in range(1, 3 * H + 1)]
        for p in range(P):
            steps = [t + 1 for t, q in enumerate(hits) if q == p]
            assert len(steps) == 3 and all(b - a == H for a, b in zip(steps, steps[1:]))   # each fragment every H steps
        assert sum(q >= 0 for q in hits) == 3 * P
        assert hits[H - 1] == P - 1                                                       # the last fragment closes the interval
    for bad in ((0, 1, 1), (5, 0, 1), (3, 4, 1), (5, 2, 0)):
        with pytest.raises(B.SlError):
            B.streaming_due(*bad)


def test_partition_by_layers_as_in_the_paper():
    from paper_2508_15706_b200.streaming import partition_by_layers
    # an 18-layer model: embedding (-1), 18 layers of 9 tensors, final norm and unembedding (layer 18)
    layers = [-1] + [l for l in range(18) for _ in range(9)] + [18, 18]
    frags = partition_by_layers(layers, 3)
    assert [len(f) for f in frags] == [1 + 54, 54, 54 + 2]
    assert frags[0][0] == 0 and frags[2][-1] == len(layers) - 1
    assert sorted(sum(frags, [])) == list(range(len(layers)))
    assert [sorted({layers[j] for j in f if 0 <= layers[j] < 18}) for f in frags] == [list(range(0, 6)), list(range(6, 12)), list(range(12, 18))]


@pytest.mark.gpu
def test_streaming_rounds_match_the_oracle():
    import torch
    import oracle as O
    from paper_2508_15706_b200 import inputs as I
    from paper_2508_15706_b200.streaming import StreamingSparseLoCo, partition_by_layers
    O.set_threads(8)
    dev = torch.device("cuda", torch.cuda.current_device())
    tensors = I.dense_transformer(128, 6, 256, 512)
    layers = [t.layer for t in tensors]
    names = [t.name for t in tensors]
    lay = [-1 if n == "embed" else (6 if n in ("final_norm", "lm_head") else l) for n, l in zip(names, layers)]
    frags = partition_by_layers(lay, 3)
    R, k, H = 2, 32, 6
    wl = I.Workload("stream", tensors, R=R, k=k, H=H, recipe="normal", seed=77, outer_lr=0.8)
    shapes, offs = [(t.rows, t.cols) for t in tensors], I.offsets(tensors)
    st = StreamingSparseLoCo(shapes, offs, frags, k=k, R=R, H=H, beta=wl.beta, outer_lr=wl.outer_lr)
    full = O.Table(shapes, offs)
    assert sum(c.payload_bytes() for c in st.ctx) == O.payload_bytes(O.Config(k=k, R=R), full)
    assert st.peak_payload_bytes() < 0.6 * O.payload_bytes(O.Config(k=k, R=R), full)
    theta = I.theta_sync(wl, dev)
    e = [I.initial_error(wl, r, dev, scale=0.5) for r in range(R)]
    th_o, e_o = theta.cpu().numpy().copy(), [x.cpu().numpy().copy() for x in e]
    cfg = O.Config(k=k, R=R, H=H, beta=wl.beta, outer_lr=wl.outer_lr)
    taken = []
    for t in range(1, 2 * H + 1):
        local = [I.theta_local(wl, theta, r, t) for r in range(R)]   # stands in for the inner step's result
        p = st.after_inner_step(t, theta, local, e)
        if p is None:
            continue
        taken.append(p)
        sub = O.Table([shapes[j] for j in frags[p]], [offs[j] for j in frags[p]])
        O.outer_step(cfg, sub, th_o, [x.cpu().numpy() for x in local], e_o)
        torch.cuda.synchronize()
        for r in range(R):
            assert np.array_equal(e[r].cpu().numpy().view(np.uint32), e_o[r].view(np.uint32)), (t, p, r)
        got = theta.cpu().numpy()
        assert np.max(np.abs(got.astype(np.float64) - th_o.astype(np.float64))) <= 1e-6 * float(np.sqrt(np.mean(th_o.astype(np.float64) ** 2)))
        theta.copy_(torch.from_numpy(th_o))
    assert taken == [0, 1, 2, 0, 1, 2]
