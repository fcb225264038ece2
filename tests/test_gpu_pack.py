"""GPU parity: projection / quantise / pack kernel against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

PATTERNS = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8), (4, 4)]


def _check(W, U, n, m, bits):
    from gpu_util import gpu_project_pack
    v, meta, s, rc = gpu_project_pack(W, U, n, m, bits)
    v_ref, meta_ref, s_ref = oracle.project_pack(W, U, n, m, bits)
    assert rc == 0
    assert np.array_equal(s, s_ref), "scales differ"
    assert np.array_equal(v, v_ref), f"values differ in {(v != v_ref).sum()} bytes"
    if n != m:
        assert np.array_equal(meta, meta_ref), "metadata differs"


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_pack_bert_rows(n, m, bits):
    # rows of 1024 (one warp per row) and 4096 (four warps per row), with the ADMM dual added
    oracle.set_threads(oracle.max_threads())
    for seed, (out, k) in enumerate([(260, 1024), (70, 4096), (133, 768), (37, 3072)]):
        W, U = wl.pack_sweep_matrix(3, seed, out, k)
        _check(W, U, n, m, bits)


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_pack_ragged_and_ties(n, m, bits):
    # widths that are not multiples of 32 / 1024 (ragged lane and chunk tails), tie-heavy grids,
    # outliers, all-zero rows and groups, and no dual
    for seed, (out, k) in enumerate([(5, 8), (3, 40), (9, 1032), (6, 2072), (4, 5000 // 8 * 8), (2, 8200)]):
        if (k // m * n * bits) % 8:
            k *= 2  # a row of packed values must be a whole number of bytes
        _check(wl.tie_heavy(100 + seed, out, k), None, n, m, bits)
        _check(wl.with_outliers(110 + seed, out, k), wl.tie_heavy(120 + seed, out, k, levels=1), n, m, bits)


def test_pack_reprojection_of_quantised_weights():
    # re-projecting dequantised weights hits exact ties and exact grid points
    W = wl.normal(np.random.default_rng(130), (64, 1024), 0.02)
    for n, m, bits in [(2, 4, 8), (2, 4, 4), (4, 8, 4)]:
        v, meta, s = oracle.project_pack(W, None, n, m, bits)
        Z = s[:, None] * oracle.unpack(v, meta, 64, 1024, n, m, bits).astype(np.float32)
        _check(Z, None, n, m, bits)


def test_pack_wide_rows():
    # 8 to 32 warps per row
    for out, k in [(3, 8192), (2, 16384 + 64), (2, 32768)]:
        W = wl.normal(np.random.default_rng(k), (out, k), 0.02)
        _check(W, None, 2, 4, 8)
        _check(W, None, 4, 8, 4)


@pytest.mark.parametrize("repeat", [1, 3])
def test_pack_batched_matches_single(repeat):
    # up to eight matrices per kernel variant travel in the kernel's parameters (repeat = 1); more go through the
    # job table in the workspace (repeat = 3: twelve matrices share the 128-thread variant)
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    shapes = [(96, 1024), (40, 4096), (64, 1024), (8, 8192), (50, 768)] * repeat
    for n, m, bits in [(2, 4, 8), (1, 4, 4)]:
        jobs, refs = [], []
        for i, (out, k) in enumerate(shapes):
            W, U = wl.pack_sweep_matrix(7, i, out, k)
            vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
            bufs = (torch.zeros(vb, dtype=torch.uint8, device=DEV), torch.zeros(mb // 4, dtype=torch.int32, device=DEV),
                    torch.zeros(out, dtype=torch.float32, device=DEV))
            jobs.append((to_dev(W), to_dev(U) if i % 2 == 0 else None, n, m, bits, *bufs))
            refs.append(oracle.project_pack(W, U if i % 2 == 0 else None, n, m, bits))
        arr = nm.make_pack_jobs(jobs)
        ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        nm.nm_project_pack_batched(arr, len(jobs), ws, ws_bytes, status)
        assert nm.nm_poll_status(status) == 0
        for job, (v_ref, m_ref, s_ref) in zip(jobs, refs):
            assert np.array_equal(job[5].cpu().numpy().reshape(v_ref.shape), v_ref)
            assert np.array_equal(job[6].cpu().numpy().view(np.uint32).reshape(m_ref.shape), m_ref)
            assert np.array_equal(job[7].cpu().numpy(), s_ref)


# one encoder's six components per configuration row, as in the paper's Table 4: Q4 / Q8 dense, S4 / S8 2:4 sparse
_TABLE4_STYLE = {"Q4": (4, 4, 4), "Q8": (4, 4, 8), "S4": (2, 4, 4), "S8": (2, 4, 8), "T8": (1, 4, 8), "E4": (4, 8, 4), "P8": (2, 8, 8)}


@pytest.mark.parametrize("layers", [1, 4])
def test_pack_batched_whole_model_to_a_heterogeneous_configuration(layers):
    """The search's inner step (Sec. 4, Eq. 6): every matrix of an encoder stack projected to its component's own
    (n, m, bits) in ONE call.  layers = 1: at most eight matrices share a kernel variant (job tables in the kernel's
    parameters); layers = 4: 24 matrices, several variants with more than eight jobs each (job table in the
    workspace), variants with a single job, and all of it in one launch sequence.  Bit for bit against the oracle."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    oracle.set_threads(oracle.max_threads())
    hidden = 256  # small hidden size, BERT's component shapes: Q, K, V, attention output h x h, FFN1 4h x h, FFN2 h x 4h
    shapes = [(hidden, hidden)] * 4 + [(4 * hidden, hidden), (hidden, 4 * hidden)]
    per_layer = [["S8", "S8", "Q8", "Q4", "S4", "S4"], ["Q8", "T8", "S8", "S8", "E4", "P8"],
                 ["S4", "S4", "S4", "Q8", "S8", "Q4"], ["S8", "Q8", "S8", "S8", "S8", "S8"]]
    jobs, refs = [], []
    for layer in range(layers):
        for comp, (out, k) in enumerate(shapes):
            n, m, bits = _TABLE4_STYLE[per_layer[layer][comp]]
            W, U = wl.pack_sweep_matrix(40 + layer, comp, out, k)
            vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
            bufs = (torch.zeros(vb, dtype=torch.uint8, device=DEV), torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV),
                    torch.zeros(out, dtype=torch.float32, device=DEV))
            jobs.append((to_dev(W), to_dev(U), n, m, bits, bufs[0], bufs[1] if mb else None, bufs[2]))
            refs.append(oracle.project_pack(W, U, n, m, bits))
    ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_project_pack_batched(nm.make_pack_jobs(jobs), len(jobs), ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == 0
    for i, (job, (v_ref, m_ref, s_ref)) in enumerate(zip(jobs, refs)):
        assert np.array_equal(job[5].cpu().numpy().reshape(v_ref.shape), v_ref), f"job {i}: values"
        if job[6] is not None:
            assert np.array_equal(job[6].cpu().numpy().view(np.uint32).reshape(m_ref.shape), m_ref), f"job {i}: metadata"
        assert np.array_equal(job[7].cpu().numpy(), s_ref), f"job {i}: scales"


def test_batched_call_with_uploaded_job_table_refuses_stream_capture():
    """More than eight jobs per kernel variant need the job table copied from host memory that lives only until the
    call returns: under stream capture the call must refuse (a replayed graph would read freed memory) and enqueue
    nothing.  The capture is ended without ever launching the graph."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    jobs = []
    for i in range(10):
        W, U = wl.pack_sweep_matrix(50, i, 16, 256)
        vb, mb = nm.nm_packed_sizes(16, 256, 2, 4, 8)
        jobs.append((to_dev(W), to_dev(U), 2, 4, 8, torch.zeros(vb, dtype=torch.uint8, device=DEV),
                     torch.zeros(mb // 4, dtype=torch.int32, device=DEV), torch.zeros(16, dtype=torch.float32, device=DEV)))
    arr = nm.make_pack_jobs(jobs)
    ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        graph.capture_begin()
        try:
            with pytest.raises(nm.NmError) as e:
                nm.nm_project_pack_batched(arr, len(jobs), ws, ws_bytes, None, stream=stream.cuda_stream)
            assert e.value.code == nm.NM_ERR_UNSUPPORTED
            # eight jobs travel in the kernel's parameters: capturing that call is fine
            nm.nm_project_pack_batched(nm.make_pack_jobs(jobs[:8]), 8, ws, ws_bytes, None, stream=stream.cuda_stream)
        finally:
            graph.capture_end()
    torch.cuda.synchronize()
    assert not jobs[0][5].any(), "the refused call, or the capture itself, ran a kernel"
    # outside capture the same call works
    nm.nm_project_pack_batched(arr, len(jobs), ws, ws_bytes, None)
    assert nm.nm_poll_status() == 0 and jobs[9][5].any()


def test_pack_flags_nonfinite_and_rejects_bad_arguments():
    import paper_2206_15014_b200 as nm
    from gpu_util import gpu_project_pack, DEV
    W = np.ones((4, 64), np.float32)
    W[2, 5] = np.nan
    assert gpu_project_pack(W, None, 2, 4, 8)[3] == nm.NM_ERR_NONFINITE
    W[2, 5] = -np.inf
    assert gpu_project_pack(W, None, 2, 4, 8)[3] == nm.NM_ERR_NONFINITE
    t = torch.zeros(64, dtype=torch.float32, device=DEV)
    for args, code in [((4, 6, 2, 4, 8), nm.NM_ERR_SHAPE), ((4, 8, 3, 4, 8), nm.NM_ERR_UNSUPPORTED),
                       ((4, 8, 2, 4, 5), nm.NM_ERR_UNSUPPORTED), ((4, 8, 5, 4, 8), nm.NM_ERR_SHAPE),
                       ((1, 65536, 2, 4, 8), nm.NM_ERR_UNSUPPORTED)]:
        with pytest.raises(nm.NmError) as e:
            nm.nm_project_pack(t, None, *args, t, t, t)
        assert e.value.code == code
    with pytest.raises(nm.NmError) as e:
        nm.nm_project_pack(t[1:], None, 2, 8, 2, 4, 8, t, t, t)
    assert e.value.code == nm.NM_ERR_ALIGN
    # empty matrix: nothing to do
    nm.nm_project_pack(t, None, 0, 8, 2, 4, 8, t, t, t)


def test_pack_is_deterministic():
    from gpu_util import gpu_project_pack
    W, U = wl.pack_sweep_matrix(3, 1, 300, 1024)
    a = gpu_project_pack(W, U, 2, 4, 8)
    b = gpu_project_pack(W, U, 2, 4, 8)
    assert all(np.array_equal(x, y) for x, y in zip(a[:3], b[:3]))


def test_activation_quantiser_matches_oracle():
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    for shape in [(128, 768), (7, 33), (1, 3), (300, 1024)]:
        Y = wl.normal(np.random.default_rng(sum(shape)), shape)
        Xq_ref, sx_ref = oracle.quantize_act(Y)
        Yd = to_dev(Y)
        amax = torch.zeros(1, dtype=torch.float32, device=DEV)
        sx = torch.zeros(1, dtype=torch.float32, device=DEV)
        Xq = torch.full((Y.size + 16,), 99, dtype=torch.int8, device=DEV)
        nm.nm_absmax(Yd, Y.size, amax)
        nm.nm_quantize_act(Yd, Y.size, amax, Xq, sx)
        assert nm.nm_poll_status() == 0
        assert sx.item() == sx_ref
        assert amax.item() == np.abs(Y).max()
        got = Xq.cpu().numpy()
        assert np.array_equal(got[:Y.size].reshape(shape), Xq_ref)
        assert (got[Y.size:] == 99).all()
    Z = torch.zeros(64, dtype=torch.float32, device=DEV)
    amax = torch.zeros(1, dtype=torch.float32, device=DEV)
    Xq = torch.ones(64, dtype=torch.int8, device=DEV)
    sx = torch.zeros(1, dtype=torch.float32, device=DEV)
    nm.nm_absmax(Z, 64, amax)
    nm.nm_quantize_act(Z, 64, amax, Xq, sx)
    assert amax.item() == 0.0 and sx.item() == 1.0 and not Xq.cpu().numpy().any()   # all-zero tensor: scale 1
    # the scale may not be written over the maximum other blocks are still reading
    with pytest.raises(nm.NmError) as e:
        nm.nm_quantize_act(Z, 64, amax, Xq, amax)
    assert e.value.code == nm.NM_ERR_SHAPE
