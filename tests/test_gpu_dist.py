"""GPU parity: the ADMM-Dist scale search and the projections that use it, against the CPU oracle.

The winning candidate is decided by comparing sums of squares held in doubles.  The kernel adds them in
another order than the oracle (per lane, over the lanes, over the warps of a row), so two candidates whose
distances agree to ~1e-12 may swap; everywhere else the candidate, the scale and every packed or dense
output must be identical.  A swapped row is checked to be a valid choice (its distance is the minimum
within 1e-9) and its outputs are compared with the oracle's projection at the scale the kernel chose.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

PATTERNS = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8), (4, 4)]
REL = 1e-9


def _gpu_dist_scales(W, U, n, m, bits, ncand):
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    out, k = W.shape
    scales = torch.full((out + 1,), float("nan"), dtype=torch.float32, device=DEV)
    cand = torch.full((out + 1,), -5, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_dist_scales(to_dev(W), to_dev(U), out, k, n, m, bits, ncand, scales, cand, status)
    rc = nm.nm_poll_status(status)
    s, c = scales.cpu().numpy(), cand.cpu().numpy()
    assert np.isnan(s[out]) and c[out] == -5, "written past the last row"
    return s[:out], c[:out], rc


def _check_choice(W, U, n, m, bits, ncand, s, c):
    """The kernel's (scale, candidate) per row against the oracle's sweep; returns the number of swapped rows."""
    E, S, s_ref, c_ref = oracle.dist_search(W, U, n, m, bits, ncand)
    rows = np.arange(W.shape[0])
    assert ((c >= 0) & (c < ncand)).all()
    assert np.array_equal(s, S[rows, c]), "scale is not the chosen candidate's"
    diff = np.nonzero(c != c_ref)[0]
    for r in diff:  # only allowed where the two distances agree to rounding
        assert E[r, c[r]] <= E[r, c_ref[r]] * (1 + REL), f"row {r}: candidate {c[r]} is not a minimiser"
    assert len(diff) <= max(1, W.shape[0] // 200), f"{len(diff)} rows differ from the oracle's choice"
    return len(diff)


def _gpu_pack_dist(W, U, n, m, bits, ncand):
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    out, k = W.shape
    vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
    values = torch.full((vb + 64,), 0xAB, dtype=torch.uint8, device=DEV)
    meta = torch.full((max(mb // 4, 1) + 16,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
    scales = torch.zeros(out, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_project_pack_dist(to_dev(W), to_dev(U), out, k, n, m, bits, ncand, values, meta if mb else None, scales, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    v, mt = values.cpu().numpy(), meta.cpu().numpy().view(np.uint32)
    assert (v[vb:] == 0xAB).all() and (mt[mb // 4:] == 0x5A5A5A5A).all(), "written past the end"
    return v[:vb].reshape(out, -1), mt[: mb // 4].reshape(out, -1) if mb else mt[:0].reshape(out, 0), scales.cpu().numpy()


def _check_pack(W, U, n, m, bits, ncand):
    v, mt, s = _gpu_pack_dist(W, U, n, m, bits, ncand)
    v_ref, m_ref, s_ref = oracle.project_pack_dist(W, U, n, m, bits, ncand)
    if not np.array_equal(s, s_ref):  # a swapped near-tie: validate the choice, then compare at the kernel's scales
        E, S, _, c_ref = oracle.dist_search(W, U, n, m, bits, ncand)
        for r in np.nonzero(s != s_ref)[0]:
            j = np.nonzero(S[r] == s[r])[0]
            assert len(j) and E[r, j[0]] <= E[r, c_ref[r]] * (1 + REL)
        assert (s != s_ref).sum() <= max(1, W.shape[0] // 200)
        v_ref, m_ref, _ = oracle.project_pack_scaled(W, U, n, m, bits, s)
    assert np.array_equal(v, v_ref), f"values differ in {(v != v_ref).sum()} bytes"
    if n != m:
        assert np.array_equal(mt, m_ref)


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_dist_scales_bert_rows(n, m, bits):
    oracle.set_threads(oracle.max_threads())
    for i, (out, k) in enumerate([(260, 1024), (70, 4096), (133, 768), (37, 3072)]):
        W, U = wl.pack_sweep_matrix(7, i, out, k)
        s, c, rc = _gpu_dist_scales(W, U, n, m, bits, 32)
        assert rc == 0
        _check_choice(W, U, n, m, bits, 32, s, c)


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_project_pack_dist_matches_oracle(n, m, bits):
    oracle.set_threads(oracle.max_threads())
    for i, (out, k) in enumerate([(200, 1024), (50, 4096), (65, 768)]):
        W, U = wl.pack_sweep_matrix(8, i, out, k)
        _check_pack(W, U, n, m, bits, 32)


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_dist_ragged_ties_outliers_and_wide_rows(n, m, bits):
    oracle.set_threads(oracle.max_threads())
    for i, (out, k) in enumerate([(5, 8), (3, 40), (9, 1032), (6, 2072), (2, 8200), (2, 16384 + 64)]):
        if (k // m * n * bits) % 8:
            k *= 2
        for W, U in ((wl.with_outliers(310 + i, out, k), wl.tie_heavy(320 + i, out, k, levels=1)),
                     (wl.tie_heavy(300 + i, out, k), None)):
            for ncand in (32, 5):
                s, c, rc = _gpu_dist_scales(W, U, n, m, bits, ncand)
                assert rc == 0
                _check_choice(W, U, n, m, bits, ncand, s, c)
            _check_pack(W, U, n, m, bits, 32)


def test_one_candidate_is_admm_max_and_extreme_magnitudes():
    from gpu_util import gpu_project_pack
    W, U = wl.pack_sweep_matrix(9, 0, 64, 1024)
    v, mt, s = _gpu_pack_dist(W, U, 2, 4, 8, 1)
    v0, m0, s0, rc = gpu_project_pack(W, U, 2, 4, 8)
    assert rc == 0 and np.array_equal(v, v0) and np.array_equal(mt, m0) and np.array_equal(s, s0)
    # scales near the ends of the fp32 range leave the reciprocal path; an all-zero matrix picks candidate 0
    for f in (np.float32(2.0 ** -125), np.float32(2.0 ** 120), np.float32(0.0)):
        Wf = (W * np.float32(50.0) * f).astype(np.float32)
        assert np.isfinite(Wf).all()
        s, c, rc = _gpu_dist_scales(Wf, None, 2, 4, 4, 32)
        assert rc == 0
        _check_choice(Wf, None, 2, 4, 4, 32, s, c)
        if f == 0:
            assert (c == 0).all() and (s == 1.0).all()


@pytest.mark.parametrize("n,m,bits", [(2, 4, 4), (1, 4, 8), (4, 8, 4), (4, 4, 4)])
def test_admm_step_dist_dense_outputs(n, m, bits):
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    oracle.set_threads(oracle.max_threads())
    for i, (out, k) in enumerate([(130, 1024), (33, 4096)]):
        W, U = wl.pack_sweep_matrix(10, i, out, k)
        Z = torch.full((out + 1, k), float("nan"), dtype=torch.float32, device=DEV)
        Un = torch.full((out + 1, k), float("nan"), dtype=torch.float32, device=DEV)
        scales = torch.zeros(out, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        nm.nm_admm_project_dist(to_dev(W), to_dev(U), out, k, n, m, bits, 32, Z, Un, None, None, scales, status)
        assert nm.nm_poll_status(status) == nm.NM_OK
        Zr, Unr, sr = oracle.admm_step_dist(W, U, n, m, bits, 32)
        assert np.array_equal(scales.cpu().numpy(), sr), "a near-tie swapped: pick another seed and report"
        Zh, Uh = Z.cpu().numpy(), Un.cpu().numpy()
        assert np.isnan(Zh[out]).all() and np.isnan(Uh[out]).all()
        assert np.array_equal(Zh[:out], Zr) and np.array_equal(Uh[:out], Unr)


def test_dist_batched_matches_single_calls_and_argument_errors():
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    specs = [(96, 1024, 2, 4, 4), (40, 4096, 2, 4, 4), (50, 768, 1, 4, 8), (8, 8192, 2, 4, 4), (30, 1024, 4, 8, 4)]
    jobs, singles = [], []
    for i, (out, k, n, m, bits) in enumerate(specs):
        W, U = wl.pack_sweep_matrix(11, i, out, k)
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        bufs = lambda: (torch.zeros(vb, dtype=torch.uint8, device=DEV), torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV),
                        torch.zeros(out, dtype=torch.float32, device=DEV))
        Wd, Ud = to_dev(W), to_dev(U)
        a, b = bufs(), bufs()
        jobs.append((Wd, Ud, n, m, bits) + a)
        nm.nm_project_pack_dist(Wd, Ud, out, k, n, m, bits, 32, *b)
        singles.append(b)
    ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_project_pack_dist_batched(nm.make_pack_jobs(jobs), len(jobs), 32, ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    for j, b in zip(jobs, singles):
        for x, y in zip(j[5:], b):
            assert torch.equal(x, y)
        assert j[5].any()
    W = to_dev(wl.pack_sweep_matrix(11, 0, 8, 64)[0])
    s = torch.zeros(8, dtype=torch.float32, device=DEV)
    for bad in (0, 33, -1):
        with pytest.raises(nm.NmError) as e:
            nm.nm_dist_scales(W, None, 8, 64, 2, 4, 8, bad, s)
        assert e.value.code == nm.NM_ERR_SHAPE
    with pytest.raises(nm.NmError):
        nm.nm_dist_scales(W, None, 8, 64, 2, 4, 8, 4, None)
    nm.nm_dist_scales(W, None, 0, 64, 2, 4, 8, 4, s)  # nothing to do


def test_admm_dist_batched_matches_oracle():
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    oracle.set_threads(oracle.max_threads())
    specs = [(64, 1024, 2, 4, 4), (20, 4096, 2, 4, 4), (33, 768, 1, 4, 8), (40, 1024, 2, 4, 4)]
    jobs, refs = [], []
    for i, (out, k, n, m, bits) in enumerate(specs):
        W, U = wl.pack_sweep_matrix(12, i, out, k)
        Wd, Ud = to_dev(W), to_dev(U)
        Z = torch.full((out, k), float("nan"), dtype=torch.float32, device=DEV)
        sc = torch.zeros(out, dtype=torch.float32, device=DEV)
        jobs.append((Wd, Ud, n, m, bits, Z, Ud, None, None, sc))          # the dual is updated in place
        refs.append(oracle.admm_step_dist(W, U, n, m, bits, 32))
    ws_bytes = nm.nm_admm_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_admm_project_dist_batched(nm.make_admm_jobs(jobs), len(jobs), 32, ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    for j, (Zr, Ur, sr) in zip(jobs, refs):
        assert np.array_equal(j[9].cpu().numpy(), sr)
        assert np.array_equal(j[5].cpu().numpy(), Zr) and np.array_equal(j[6].cpu().numpy(), Ur)
    with pytest.raises(nm.NmError):
        nm.nm_admm_project_dist_batched(nm.make_admm_jobs(jobs), len(jobs), 0, ws, ws_bytes, status)
