"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.
Bit-exact payloads (indices, codes, tables) and error buffers; theta_sync within 1e-6 x RMS."""
import numpy as np
import pytest
import torch

from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _case(*a, **kw):
    from parity import DeviceCase, oracle_threads
    oracle_threads()
    return DeviceCase(*a, **kw)


SMALL = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("flat", 1, 5000, 0), I.TensorSpec("router", 8, 1024, 1),
         I.TensorSpec("norm", 1, 768, 1), I.TensorSpec("tiny", 1, 40, 2), I.TensorSpec("odd2d", 70, 64, 2),
         I.TensorSpec("mid", 1, 4096 + 2051, 3), I.TensorSpec("b", 64, 64, 3)]


def test_config1_single_tensor_with_ties():
    wl = I.workload("c1_single_1024")
    c = _case(wl)
    for step in range(2):
        c.fill_local(step)
        snap = c.snapshot([0])
        c.step()
        rep = c.check(snap)
        assert rep["tensors"] == 1
    assert c.sl.payload_bytes() == 28688


@pytest.mark.parametrize("k", [1, 41, 64, 82, 123, 256])
def test_small_shapes_k_sweep(k):
    wl = I.Workload("small", SMALL, R=3, k=k, recipe="student_t4", seed=20 + k, outer_lr=0.7)
    c = _case(wl, e_scale=0.5)
    for step in range(2):
        c.fill_local(step)
        snap = c.snapshot(range(len(SMALL)))
        c.step()
        c.check(snap)


def test_zero_and_heavy_ties():
    wl = I.Workload("ties", SMALL, R=2, k=64, recipe="normal", seed=31)
    c = _case(wl)
    g = torch.Generator(device="cpu").manual_seed(5)
    n = c.theta.numel()
    # worker 0: theta_local == theta_sync and e == 0  -> all-zero chunks
    c.local[0].copy_(c.theta)
    # worker 1: drift takes five magnitudes only (both signs) -> every chunk is one big tie group
    vals = torch.tensor([0.0, 2.0 ** -9, -2.0 ** -9, 2.0 ** -7, -2.0 ** -7], dtype=torch.float32)
    pick = vals[torch.randint(0, 5, (n,), generator=g)].to(c.dev)
    c.theta.copy_(torch.round(c.theta * 1024) / 1024)  # exact differences
    c.local[0].copy_(c.theta)
    c.local[1].copy_(c.theta - pick)
    snap = c.snapshot(range(len(SMALL)))
    c.step()
    c.check(snap)
    # second step: zero drift with non-zero error buffers
    c.local[1].copy_(c.theta)
    c.local[0].copy_(c.theta)
    snap = c.snapshot(range(len(SMALL)))
    c.step()
    c.check(snap)


def test_extreme_values():
    """Denormals are ordinary values: nothing is flushed to zero on either side."""
    wl = I.Workload("extreme", [I.TensorSpec("a", 64, 128, 0), I.TensorSpec("v", 1, 4096, 0)], R=1, k=64,
                    recipe="normal", seed=33, beta=1.0)
    c = _case(wl)
    c.fill_local(0)
    n = c.theta.numel()
    g = torch.Generator(device="cpu").manual_seed(6)
    pos = torch.randperm(n, generator=g)[:600].to(c.dev)
    c.theta[pos[:200]] = 0.0
    c.local[0][pos[:100]] = 1e-41
    c.local[0][pos[100:200]] = -3e-42
    c.e[0][pos[200:400]] = 2e-44
    c.local[0][pos[400:600]] = c.theta[pos[400:600]]
    snap = c.snapshot([0, 1])
    c.step()
    c.check(snap)


def test_error_feedback_freeze():
    wl = I.Workload("freeze", SMALL, R=2, k=64, recipe="normal", seed=41)
    c = _case(wl, e_scale=0.5)
    c.sl.set_hyper(ef_enabled=False)
    c.fill_local(0)
    e_before = [x.clone() for x in c.e]
    snap = c.snapshot(range(len(SMALL)))
    c.step()
    c.check(snap, ef_enabled=False)
    for a, b in zip(c.e, e_before):
        assert torch.equal(a, b)


@pytest.mark.parametrize("k", [41, 64, 200])
def test_deferred_subtraction_is_bit_identical(k):
    """Deferred error-feedback subtraction: payloads, theta_sync and the true error buffers match the
    oracle after every step, through a frozen step (which writes the waiting values out first), and
    the buffers themselves hold the true error after a flush."""
    wl = I.Workload("deferred", SMALL, R=3, k=k, recipe="student_t4", seed=90 + k, outer_lr=0.9)
    c = _case(wl, e_scale=0.5)
    c.sl.set_ef_deferred(True)
    for step in range(5):
        frozen = step == 3
        c.sl.set_hyper(ef_enabled=not frozen)
        c.fill_local(step)
        snap = c.snapshot(range(len(SMALL)))
        c.step()
        assert c.sl.ef_pending() == (not frozen)
        c.check(snap, ef_enabled=not frozen)
    assert c.sl.ef_pending()
    want = [x.clone() for x in c.true_error()]
    c.sl.ef_flush()
    torch.cuda.synchronize()
    assert not c.sl.ef_pending()
    for a, b in zip(c.e, want):
        assert torch.equal(a, b)
    # pointers of other buffers are refused while values wait
    c.fill_local(9)
    c.step()
    from paper_2508_15706_b200 import binding as B
    with pytest.raises(B.SlError) as ei:
        c.sl.outer_step(c.theta, [c.local_of(r) for r in range(3)], [x.clone() for x in c.e], c.payloads)
    assert ei.value.status == B.SL_ERR_INVALID_ARG
    # a default-mode twin ends in the same state
    d = _case(wl, e_scale=0.5)
    c2 = _case(wl, e_scale=0.5)
    c2.sl.set_ef_deferred(True)
    for step in range(3):
        for x in (d, c2):
            x.fill_local(step)
            x.step()
    c2.sl.ef_flush()
    torch.cuda.synchronize()
    assert torch.equal(d.theta, c2.theta)
    for r in range(3):
        assert torch.equal(d.e[r], c2.e[r]) and torch.equal(d.payloads[r], c2.payloads[r])


ALIGNED = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("flat", 1, 4096 * 2 + 1024, 0), I.TensorSpec("wide", 64, 512, 1),
           I.TensorSpec("norm", 1, 768, 1), I.TensorSpec("b", 192, 64, 2), I.TensorSpec("tail", 1, 4096 + 64 * 7, 2)]


@pytest.mark.parametrize("deferred", [False, True])
def test_tensor_map_copies_match_oracle_and_per_thread_copies(deferred):
    """A table whose blocks all start on 64-element boundaries takes the tensor-map (TMA) block copies;
    the same steps with the per-thread copies must give the same bits, and both match the oracle."""
    from paper_2508_15706_b200 import binding as B
    wl = I.Workload("aligned", ALIGNED, R=3, k=64, recipe="student_t4", seed=77, outer_lr=0.9)
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    a.sl.set_tile_copies(True)    # raises if the table were not eligible
    b.sl.set_tile_copies(False)
    for c in (a, b):
        c.sl.set_ef_deferred(deferred)
    for step in range(3):
        for c in (a, b):
            c.fill_local(step)
        snap = a.snapshot(range(len(ALIGNED)))
        a.step()
        b.step()
        a.check(snap)
        assert torch.equal(a.theta, b.theta)
        for r in range(3):
            assert torch.equal(a.payloads[r], b.payloads[r])
    ea, eb = a.true_error(), b.true_error()
    torch.cuda.synchronize()
    for x, y in zip(ea, eb):
        assert torch.equal(x, y)
    # a table with an odd offset cannot use block copies
    sl = B.SparseLoCo([(1, 100), (64, 64)], k=8, R=1)
    with pytest.raises(B.SlError) as ei:
        sl.set_tile_copies(True)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED


@pytest.mark.parametrize("R,deferred", [(1, True), (1, False), (40, True), (64, False)])
def test_worker_count_extremes(R, deferred):
    """One worker (every unit starts a new chunk) and more than 32 workers (the apply kernel takes them
    in two batches), on a table that takes the tensor-map copies."""
    wl = I.Workload("extremes", ALIGNED, R=R, k=64, recipe="normal", seed=300 + R, outer_lr=0.8)
    c = _case(wl, e_scale=0.5, distinct_local=min(R, 4))
    c.sl.set_ef_deferred(deferred)
    for step in range(2):
        c.fill_local(step)
        snap = c.snapshot(range(len(ALIGNED)))
        c.step()
        c.check(snap)


def test_sl_compress_on_an_aligned_table_matches_outer_step():
    """sl_compress (one worker, tensor-map copies) leaves what sl_outer_step leaves for that worker."""
    wl = I.Workload("single", ALIGNED, R=2, k=41, recipe="student_t4", seed=321)
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    for step in range(2):
        a.fill_local(step)
        b.fill_local(step)
        a.step()
        for r in range(2):
            b.sl.compress(b.theta, b.local[r], b.e[r], b.payloads[r])
        b.sl.aggregate_apply(b.payloads, b.theta)
        torch.cuda.synchronize()
        assert b.sl.device_status() == 0
        assert torch.equal(a.theta, b.theta)
        for r in range(2):
            assert torch.equal(a.e[r], b.e[r]) and torch.equal(a.payloads[r], b.payloads[r])


def test_tensor_map_table_survives_many_buffers():
    """Every new buffer pointer gets tensor maps on first use; the table of maps is finite, so a caller
    that keeps passing fresh buffers makes it start over.  Results must not care."""
    wl = I.Workload("slots", ALIGNED, R=3, k=64, recipe="normal", seed=430)
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    b.sl.set_tile_copies(False)
    keep = []
    for step in range(60):   # 3 fresh theta_local buffers per step: 180 pointers > the table's capacity
        a.fill_local(step % 3)
        fresh = [x.clone() for x in a.local]
        keep.append(fresh)   # keep them alive so that the allocator cannot hand the same address out again
        a.sl.outer_step(a.theta, fresh, a.e, a.payloads)
        b.fill_local(step % 3)
        b.step()
    torch.cuda.synchronize()
    assert a.sl.device_status() == 0
    assert torch.equal(a.theta, b.theta)
    for r in range(3):
        assert torch.equal(a.e[r], b.e[r]) and torch.equal(a.payloads[r], b.payloads[r])


@pytest.mark.parametrize("buffers", [1, 2])
def test_outer_step_from_host_buffers_equals_resident_step(buffers):
    """sl_outer_step_host (workers' parameters in pinned host memory, staged through one or two device
    buffers, theta copied back) leaves the same bits as sl_outer_step on resident copies."""
    wl = I.Workload("host", ALIGNED, R=3, k=64, recipe="normal", seed=440, outer_lr=0.9)
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    flat = a.theta.numel()
    flat4 = (flat + 3) // 4 * 4
    stage = torch.empty(buffers * flat4, dtype=torch.float32, device=a.dev)
    theta_host = torch.empty(flat, dtype=torch.float32, pin_memory=True)
    for step in range(2):
        a.fill_local(step)
        b.fill_local(step)
        hosts = [x.cpu().pin_memory() for x in b.local]
        a.step()
        b.sl.outer_step_host(b.theta, hosts, stage, b.e, b.payloads, theta_host)
        assert b.sl.device_status() == 0
        assert torch.equal(a.theta, b.theta) and torch.equal(theta_host, b.theta.cpu())
        for r in range(3):
            assert torch.equal(a.e[r], b.e[r]) and torch.equal(a.payloads[r], b.payloads[r])


def test_side_stream_gives_the_same_result():
    """All work (kernels, tensor-map uploads, memsets) is ordered on the caller's stream: steps issued
    on a side stream without host synchronisation in between match steps on the default stream."""
    wl = I.Workload("stream", ALIGNED, R=3, k=64, recipe="normal", seed=450)
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    for c in (a, b):
        c.sl.set_ef_deferred(True)
        c.fill_local(0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    for step in range(4):
        a.sl.outer_step(a.theta, a.local, a.e, a.payloads)
    with torch.cuda.stream(side):
        for step in range(4):
            b.sl.outer_step(b.theta, b.local, b.e, b.payloads)
        b.sl.ef_flush()
    a.sl.ef_flush()
    side.synchronize()
    torch.cuda.synchronize()
    assert a.sl.device_status() == 0 and b.sl.device_status() == 0
    assert torch.equal(a.theta, b.theta)
    for r in range(3):
        assert torch.equal(a.e[r], b.e[r]) and torch.equal(a.payloads[r], b.payloads[r])


def test_outer_step_in_a_cuda_graph():
    """No entry point synchronises the host, so a step can be captured in a CUDA graph (after one
    eager call, which builds the tensor maps of the buffers) and replayed: same bits as eager steps."""
    wl = I.workload("c1_single_1024")
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    for c in (a, b):
        c.fill_local(0)
        c.step()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            a.sl.outer_step(a.theta, a.local, a.e, a.payloads)
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
        b.sl.outer_step(b.theta, b.local, b.e, b.payloads)
    torch.cuda.synchronize()
    assert a.sl.device_status() == 0
    assert torch.equal(a.theta, b.theta)
    for r in range(wl.R):
        assert torch.equal(a.e[r], b.e[r]) and torch.equal(a.payloads[r], b.payloads[r])


def test_degenerate_tensor_sizes():
    """One-element and few-element tensors (k far above the chunk length), a single row shorter than a
    vector, and a table whose only tensor is a short chunk."""
    tiny = [I.TensorSpec("one", 1, 1, 0), I.TensorSpec("three", 1, 3, 0), I.TensorSpec("col", 7, 1, 1),
            I.TensorSpec("w", 64, 64, 1), I.TensorSpec("five", 5, 5, 2)]
    for k in (1, 64, 256):
        wl = I.Workload("tiny", tiny, R=2, k=k, recipe="normal", seed=900 + k)
        c = _case(wl, e_scale=0.5)
        for step in range(2):
            c.fill_local(step)
            snap = c.snapshot(range(len(tiny)))
            c.step()
            c.check(snap)
    wl = I.Workload("lonely", [I.TensorSpec("v", 1, 100, 0)], R=1, k=64, recipe="normal", seed=950)
    c = _case(wl)
    c.fill_local(0)
    snap = c.snapshot([0])
    c.step()
    c.check(snap)


def test_fragment_contexts_equal_one_full_step():
    """Streaming (the paper's fragment-wise variant) needs nothing new: contexts over disjoint subsets
    of the tensors, with offsets into the same flat buffers, each take the outer step of their
    fragment; together they leave theta and the error buffers exactly as one step over all tensors."""
    from paper_2508_15706_b200.binding import SparseLoCo
    wl = I.Workload("fragments", ALIGNED, R=3, k=64, recipe="normal", seed=410, outer_lr=0.8)
    full = _case(wl, e_scale=0.5)
    frag = _case(wl, e_scale=0.5)
    full.fill_local(0)
    frag.fill_local(0)
    full.step()
    ids = [[0, 1, 2], [3, 4, 5]]
    for sub in ids:
        sl = SparseLoCo([full.shapes[j] for j in sub], [full.offs[j] for j in sub], k=64, R=3, beta=wl.beta,
                        outer_lr=wl.outer_lr)
        pays = [torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=frag.dev) for _ in range(3)]
        sl.outer_step(frag.theta, frag.local, frag.e, pays)
        torch.cuda.synchronize()
        assert sl.device_status() == 0
    assert torch.equal(full.theta, frag.theta)
    for r in range(3):
        assert torch.equal(full.e[r], frag.e[r])


def test_compress_then_aggregate_equals_outer_step_and_absent_workers():
    import oracle as O
    wl = I.Workload("split", SMALL, R=3, k=64, recipe="normal", seed=51, outer_lr=0.8)
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    a.fill_local(0)
    b.fill_local(0)
    a.step()
    for r in range(3):
        b.sl.compress(b.theta, b.local[r], b.e[r], b.payloads[r])
    theta_before = b.theta.clone()
    b.sl.aggregate_apply(b.payloads, b.theta)
    torch.cuda.synchronize()
    assert torch.equal(a.theta, b.theta)
    for r in range(3):
        assert torch.equal(a.e[r], b.e[r]) and torch.equal(a.payloads[r], b.payloads[r])
    # one worker absent: oracle with the same payloads, divisor R then divisor 2
    pays = [p.cpu().numpy() for p in b.payloads]
    tab = O.Table(b.shapes, b.offs)
    for dbp in (0, 1):
        th = theta_before.clone()
        b.sl.set_hyper(divide_by_present=bool(dbp))
        b.sl.aggregate_apply([b.payloads[0], None, b.payloads[2]], th)
        th_o = theta_before.cpu().numpy().copy()
        O.aggregate_apply(O.Config(k=64, R=3, outer_lr=0.8, divide_by_present=dbp), tab, [pays[0], None, pays[2]], th_o)
        rms = float(np.sqrt(np.mean(th_o.astype(np.float64) ** 2)))
        assert np.max(np.abs(th.cpu().numpy().astype(np.float64) - th_o)) <= 1e-6 * rms
    # nobody present: theta untouched
    th = theta_before.clone()
    b.sl.aggregate_apply([None, None, None], th)
    torch.cuda.synchronize()
    assert torch.equal(th, theta_before)


def test_runs_are_bit_reproducible():
    wl = I.Workload("repro", SMALL, R=4, k=64, recipe="student_t4", seed=61)
    outs = []
    for _ in range(2):
        c = _case(wl, e_scale=0.5)
        c.fill_local(0)
        c.step()
        torch.cuda.synchronize()
        outs.append((c.theta.clone(), [x.clone() for x in c.e], [p.clone() for p in c.payloads]))
    assert torch.equal(outs[0][0], outs[1][0])
    for x, y in zip(outs[0][1] + outs[0][2], outs[1][1] + outs[1][2]):
        assert torch.equal(x, y)


@pytest.mark.parametrize("bits,k", [(2, 41), (1, 41), (3, 64), (4, 41), (2, 300), (4, 1000)])
def test_validate_payload_flags_corruption(bits, k):
    """(every quantiser width and k beyond 256 share the record layout: 12-bit indices, then the codes)"""
    wl = I.Workload("val", SMALL, R=1, k=k, recipe="normal", seed=71)
    c = _case(wl, quant_bits=bits)
    c.fill_local(0)
    c.step()
    status = torch.full((1,), -1, dtype=torch.int32, device=c.dev)
    c.sl.validate_payload(c.payloads[0], status)
    torch.cuda.synchronize()
    assert status.item() == 0
    stride = c.stride
    first = c.rec_off[0]
    corruptions = []
    p = c.payloads[0].clone()
    p[first] = 0xFF; p[first + 1] = 0xFF  # index 0xFFF first, then a smaller one: not ascending
    corruptions.append(p)
    if (12 * k + 7) // 8 + (bits * k + 7) // 8 < stride:   # (some k fill the stride exactly: no padding to spoil)
        p = c.payloads[0].clone()
        p[first + stride - 1] = 1  # padding must be zero
        corruptions.append(p)
    p = c.payloads[0].clone()
    p[0:4] = torch.tensor(np.frombuffer(np.float32(np.inf).tobytes(), np.uint8).copy())  # table not finite
    corruptions.append(p)
    p = c.payloads[0].clone()
    tiny_rec = c.rec_off[4]  # the 40-element tensor: slots >= 40 must be zero
    p[tiny_rec + (12 * 40) // 8 + 1] = 0x10
    corruptions.append(p)
    if bits == 1:  # a 1-bit table is 8 bytes of a 16-byte header: the rest must be zero
        p = c.payloads[0].clone()
        p[12] = 1
        corruptions.append(p)
    for bad in corruptions:
        c.sl.validate_payload(bad, status)
        torch.cuda.synchronize()
        assert status.item() == 4
    # a corrupted payload must not fault the apply kernel either (indices beyond the chunk are dropped)
    th = c.theta.clone()
    c.sl.aggregate_apply([corruptions[0]], th)
    torch.cuda.synchronize()


def test_argument_errors():
    from paper_2508_15706_b200 import binding as B
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo([(64, 64)], k=64, R=1, chunk_elems=1024, tile_dim=32)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo([(64, 64)], k=0, R=1)
    assert ei.value.status == B.SL_ERR_INVALID_ARG
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo([(64, 64)], k=2049, R=1)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo([(64, 64), (1, 10)], offsets=[0, 4098], k=8, R=1)
    assert ei.value.status == B.SL_ERR_ALIGNMENT
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo([(64, 64)], k=8, R=1, beta=1.5)
    assert ei.value.status == B.SL_ERR_INVALID_ARG
    sl = B.SparseLoCo([(64, 64)], k=8, R=2, alloc_workspace=False)
    dev = torch.device("cuda")
    th = torch.zeros(4096, device=dev)
    pay = [torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev) for _ in range(2)]
    e = [torch.zeros(4096, device=dev) for _ in range(2)]
    with pytest.raises(B.SlError) as ei:  # no workspace lent
        sl.outer_step(th, [th, th], e, pay)
    assert ei.value.status == B.SL_ERR_NOMEM
    ws = torch.empty(sl.workspace_bytes(), dtype=torch.uint8, device=dev)
    sl.set_workspace(ws)
    with pytest.raises(B.SlError) as ei:  # aliased error buffers
        sl.outer_step(th, [th, th], [e[0], e[0]], pay)
    assert ei.value.status == B.SL_ERR_INVALID_ARG
    with pytest.raises(B.SlError) as ei:  # misaligned pointer
        sl.outer_step(th, [th, th], e, [pay[0], pay[1][1:]])
    assert ei.value.status == B.SL_ERR_ALIGNMENT
    sl.outer_step(th, [th, th], e, pay)
    torch.cuda.synchronize()


def test_read_stats_matches_the_oracle_statistics():
    """sl_read_stats: per (worker, tensor) mean, sigma, 3 sigma and the four table entries of the last
    compression, bit for bit those of the oracle's quantiser (Sec. 4), for every worker slot; a tensor
    of more than 64 chunks takes the second summation group."""
    import oracle as O
    tensors = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("big", 576, 640, 0), I.TensorSpec("norm", 1, 768, 1),
               I.TensorSpec("flat", 1, 4096 * 2 + 100, 1)]
    wl = I.Workload("stats", tensors, R=3, k=64, recipe="student_t4", seed=91)
    c = _case(wl, e_scale=0.5)
    c.fill_local(0)
    snap = c.snapshot(range(len(tensors)))
    c.step()
    cfg = O.Config(k=wl.k, R=wl.R, beta=wl.beta, outer_lr=wl.outer_lr)
    for r in range(wl.R):
        got = c.sl.read_stats(r, len(tensors)).cpu().numpy()
        for j, t in enumerate(tensors):
            out = O.compress(cfg, O.Table([(t.rows, t.cols)]), snap[j]["theta"], snap[j]["local"][r], snap[j]["e"][r].copy())
            mu, sigma, lut = out.stats[0, 0], out.stats[0, 1], out.stats[0, 2:6]
            want = np.array([mu, sigma, np.float32(3.0) * sigma, *lut, 0.0], np.float32)
            assert np.array_equal(got[j].view(np.uint32), want.view(np.uint32)), (r, t.name, got[j], want)


def test_two_live_contexts_with_different_k():
    """Kernel attributes (the dynamic shared-memory limit) belong to the function, not to a context: a
    context created later with a smaller k must not take away what an earlier one with a larger k needs."""
    from paper_2508_15706_b200 import binding as B
    dev = torch.device("cuda", torch.cuda.current_device())
    shapes = [(128, 128), (1, 5000)]
    big = B.SparseLoCo(shapes, k=256, R=2)
    small = B.SparseLoCo(shapes, k=8, R=2)       # created after `big`
    n = big.flat_elems()
    g = torch.Generator(device=dev).manual_seed(5)
    theta = torch.randn(n, device=dev, generator=g) * 0.02
    for sl in (big, small, big):
        local = [theta - 1e-3 * torch.randn(n, device=dev, generator=g) for _ in range(2)]
        e = [torch.zeros(n, device=dev) for _ in range(2)]
        pay = [torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev) for _ in range(2)]
        sl.outer_step(theta, local, e, pay)
        sl.aggregate_apply(pay, theta)
        cap = sl.coded_payload_capacity()
        coded = torch.zeros(cap, dtype=torch.uint8, device=dev)
        size = torch.zeros(1, dtype=torch.int64, device=dev)
        sl.encode_payload(pay[0], coded, size)
        sl.aggregate_apply_coded([coded, None], theta, [int(size.item()), 0])
        torch.cuda.synchronize()
        assert sl.device_status() == 0


def test_deferred_subtraction_in_sl_compress():
    """The deployment with one worker per GPU calls sl_compress for its own worker only.  With deferral on,
    that worker's corrected values wait in the workspace for its next sl_compress: payloads must be the
    oracle's at every step, the true error (the waiting values written into a copy) too, and a call that
    cannot use them (sl_outer_step with all workers) must first put them where they belong."""
    import oracle as O
    wl = I.Workload("compress_deferred", SMALL, R=2, k=41, recipe="student_t4", seed=91)
    c = _case(wl, e_scale=0.5)
    c.sl.set_ef_deferred(True)
    tab = O.Table(c.shapes, c.offs)
    cfg = O.Config(k=41, R=2, beta=wl.beta, outer_lr=wl.outer_lr)
    theta_o = c.theta.cpu().numpy()
    e_o = c.e[0].cpu().numpy().copy()
    coded = torch.zeros(c.sl.coded_payload_capacity(), dtype=torch.uint8, device=c.dev)
    size = torch.zeros(1, dtype=torch.int64, device=c.dev)
    for step in range(3):
        c.fill_local(step)
        c.sl.compress(c.theta, c.local_of(0), c.e[0], c.payloads[0])
        torch.cuda.synchronize()
        assert c.sl.ef_pending() and c.guards_intact()
        # the wire codec borrows scratch from the workspace in which the values wait: it must not disturb them
        c.sl.encode_payload(c.payloads[0], coded, size)
        out = O.compress(cfg, tab, theta_o, c.local_of(0).cpu().numpy(), e_o)
        assert np.array_equal(c.payloads[0].cpu().numpy(), out.payload), step
        copy = c.e[0].clone()
        c.sl.ef_flush([copy], keep_pending=True)
        torch.cuda.synchronize()
        assert np.array_equal(copy.cpu().numpy().view(np.uint32), e_o.view(np.uint32)), step
        assert not np.array_equal(c.e[0].cpu().numpy().view(np.uint32), e_o.view(np.uint32))  # (they do wait)
    # a full outer step next: the single worker's values are written out before anything else happens
    c.fill_local(3)
    snap = c.snapshot(range(len(SMALL)))
    assert np.array_equal(snap[0]["e"][1], c.e[1][c.offs[0]:c.offs[0] + SMALL[0].numel].cpu().numpy())
    c.step()
    for j in snap:   # the snapshot was taken with the values still waiting: give the oracle the true error
        t, off = SMALL[j], c.offs[j]
        snap[j]["e"][0] = e_o[off:off + t.numel].copy()
    c.check(snap)
