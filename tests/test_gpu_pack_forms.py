"""GPU parity of the projection kernel's three forms in blocks of four warps, each forced in turn.

The library picks the form from the launch (dense outputs and short launches: chunks staged in shared memory
by bulk copies; long launches: chunks asked for ahead into L2; the one-unit-per-block form stays for
measurements), so the other parity tests meet mostly one of them.  Here every form runs every pattern and
code width on rows of one and four warps, ragged tails, a launch of many rounds per resident block, a batch
through the device job table, and the ADMM step with dense outputs, bit for bit against the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

PATTERNS = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8), (4, 4)]
FORMS = {"direct": 1, "staged": 2, "ahead": 3}


@pytest.fixture(params=sorted(FORMS))
def form(request):
    import paper_2206_15014_b200 as nm
    nm.nm_debug_set_option("pack_form", FORMS[request.param])
    yield request.param
    nm.nm_debug_set_option("pack_form", 0)


def _check_pack(W, U, n, m, bits):
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
def test_forms_rows_and_ragged(form, n, m, bits):
    oracle.set_threads(oracle.max_threads())
    for seed, (out, k) in enumerate([(260, 1024), (70, 4096), (37, 3072)]):
        W, U = wl.pack_sweep_matrix(3, seed, out, k)
        _check_pack(W, U, n, m, bits)
    for seed, (out, k) in enumerate([(5, 8), (9, 1032), (6, 2072)]):
        if (k // m * n * bits) % 8:
            k *= 2
        _check_pack(wl.tie_heavy(100 + seed, out, k), None, n, m, bits)
        _check_pack(wl.with_outliers(110 + seed, out, k), wl.tie_heavy(120 + seed, out, k, levels=1), n, m, bits)


@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (4, 8, 4), (1, 8, 8)])
def test_forms_many_rounds(form, n, m, bits):
    """More units than resident blocks, several times over (9001 rows of 1024: 2251 units; 1500 rows of 3072: a row
    spans four warps, one of them past the row's end), with the last block's rows running out."""
    oracle.set_threads(oracle.max_threads())
    for seed, (out, k) in enumerate([(9001, 1024), (1500, 3072)]):
        W, U = wl.pack_sweep_matrix(11, seed, out, k)
        _check_pack(W, U, n, m, bits)


def test_forms_batched_through_the_job_table(form):
    """Twelve matrices of mixed shapes in one launch (device job table): a block's consecutive units cross from one
    job into the next."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    shapes = [(96, 1024), (40, 4096), (64, 1024), (700, 1024), (50, 768), (330, 2048)] * 2
    n, m, bits = 2, 4, 8
    jobs, refs = [], []
    for i, (out, k) in enumerate(shapes):
        W, U = wl.pack_sweep_matrix(17, i, out, k)
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


@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (4, 8, 8), (1, 4, 4), (4, 4, 4)])
def test_forms_admm_step(form, n, m, bits):
    """Dense outputs (Z, U_next) besides the packed ones, 3000 rows: several rounds per resident block."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    oracle.set_threads(oracle.max_threads())
    for seed, (out, k) in enumerate([(3000, 1024), (301, 4096), (9, 1032)]):
        W, U = wl.pack_sweep_matrix(23, seed, out, k)
        Z = torch.full((out + 1, k), float("nan"), dtype=torch.float32, device=DEV)
        Un = torch.full((out + 1, k), float("nan"), dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        values = torch.zeros(vb, dtype=torch.uint8, device=DEV)
        meta = torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV)
        scales = torch.zeros(out, dtype=torch.float32, device=DEV)
        nm.nm_admm_project(to_dev(W), to_dev(U), out, k, n, m, bits, Z, Un, values, meta if n != m else None, scales,
                           status=status)
        assert nm.nm_poll_status(status) == 0
        Zh, Uh = Z.cpu().numpy(), Un.cpu().numpy()
        assert np.isnan(Zh[out]).all() and np.isnan(Uh[out]).all(), "written past the last row"
        Zr, Unr, sr = oracle.admm_step(W, U, n, m, bits)
        assert np.array_equal(Zh[:out], Zr) and np.array_equal(Uh[:out], Unr)
        v_ref, meta_ref, s_ref = oracle.project_pack(W, U, n, m, bits)
        assert np.array_equal(scales.cpu().numpy(), s_ref)
        assert np.array_equal(values.cpu().numpy(), np.asarray(v_ref).reshape(-1))
        if n != m:
            assert np.array_equal(meta.cpu().numpy().view(np.uint32)[: mb // 4], np.asarray(meta_ref).reshape(-1))
