"""GPU parity: one ADMM projection step with dense outputs (nm_admm_project) against the CPU oracle.

Z (dequantised joint projection), U_next (dual update) and the optional packed outputs are compared bit
for bit: both sides round the same operations (fp32 add, IEEE division and round-half-even inside the
quantiser, one multiply s * code, one subtract).
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

PATTERNS = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8), (4, 4)]


def _gpu_admm(W, U, n, m, bits, want_u=True, want_packed=True):
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    out, k = W.shape
    Wd, Ud = to_dev(W), to_dev(U)
    Z = torch.full((out + 1, k), float("nan"), dtype=torch.float32, device=DEV)       # one guard row
    Un = torch.full((out + 1, k), float("nan"), dtype=torch.float32, device=DEV) if want_u else None
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
    values = torch.zeros(vb, dtype=torch.uint8, device=DEV) if want_packed else None
    meta = torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV) if want_packed else None
    scales = torch.zeros(out, dtype=torch.float32, device=DEV) if want_packed else None
    nm.nm_admm_project(Wd, Ud, out, k, n, m, bits, Z, Un, values, meta if n != m else None, scales, status=status)
    rc = nm.nm_poll_status(status)
    Zh = Z.cpu().numpy()
    assert np.isnan(Zh[out]).all(), "Z written past the last row"
    Unh = None
    if want_u:
        Unh = Un.cpu().numpy()
        assert np.isnan(Unh[out]).all(), "U_next written past the last row"
        Unh = Unh[:out]
    packed = None
    if want_packed:
        packed = (values.cpu().numpy(), meta.cpu().numpy().view(np.uint32)[: mb // 4], scales.cpu().numpy())
    return Zh[:out], Unh, packed, rc


def _check(W, U, n, m, bits):
    Z, Un, packed, rc = _gpu_admm(W, U, n, m, bits)
    assert rc == 0
    Zr, Unr, sr = oracle.admm_step(W, U, n, m, bits)
    assert np.array_equal(Z, Zr), f"Z differs in {(Z != Zr).sum()} of {Z.size}"
    assert np.array_equal(Un, Unr), f"U_next differs in {(Un != Unr).sum()} of {Un.size}"
    v_ref, meta_ref, s_ref = oracle.project_pack(W, U, n, m, bits)
    assert np.array_equal(packed[2], s_ref) and np.array_equal(packed[0], np.asarray(v_ref).reshape(-1))
    if n != m:
        assert np.array_equal(packed[1], np.asarray(meta_ref).reshape(-1))


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_admm_step_bert_rows(n, m, bits):
    oracle.set_threads(oracle.max_threads())
    for seed, (out, k) in enumerate([(260, 1024), (70, 4096), (133, 768), (37, 3072)]):
        W, U = wl.pack_sweep_matrix(3, seed, out, k)
        _check(W, U, n, m, bits)


@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_admm_step_ragged_ties_and_wide_rows(n, m, bits):
    for seed, (out, k) in enumerate([(5, 8), (3, 40), (9, 1032), (6, 2072), (2, 8200), (2, 16384 + 64)]):
        if (k // m * n * bits) % 8:
            k *= 2
        _check(wl.with_outliers(210 + seed, out, k), wl.tie_heavy(220 + seed, out, k, levels=1), n, m, bits)
        _check(wl.tie_heavy(200 + seed, out, k), None, n, m, bits)


def test_ste_forward_form_and_optional_outputs():
    # no dual in, none out, no packed outputs: the fake-quantised, N:M-projected weight alone
    W = wl.normal(np.random.default_rng(230), (300, 1024), 0.02)
    Z, Un, packed, rc = _gpu_admm(W, None, 2, 4, 8, want_u=False, want_packed=False)
    assert rc == 0 and Un is None and packed is None
    Zr, _, _ = oracle.admm_step(W, None, 2, 4, 8, want_u=False)
    assert np.array_equal(Z, Zr)
    # fixed point: projecting Z again reproduces it (same codes; the scale may move by an ulp) and leaves ~0 in the dual
    Z2, U2, _, _ = _gpu_admm(Z, None, 2, 4, 8)
    Z2r, U2r, _ = oracle.admm_step(Z, None, 2, 4, 8)
    assert np.array_equal(Z2, Z2r) and np.array_equal(U2, U2r)
    assert np.all(np.abs(U2) <= np.abs(Z) * 2.0 ** -22)


def test_admm_step_in_place_dual_and_errors():
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    W, U = wl.pack_sweep_matrix(3, 7, 128, 1024)
    Wd, Ud = to_dev(W), to_dev(U)
    Z = torch.empty((128, 1024), dtype=torch.float32, device=DEV)
    nm.nm_admm_project(Wd, Ud, 128, 1024, 2, 4, 8, Z, Ud)        # U_next written over U
    torch.cuda.synchronize()
    Zr, Unr, _ = oracle.admm_step(W, U, 2, 4, 8)
    assert np.array_equal(Z.cpu().numpy(), Zr) and np.array_equal(Ud.cpu().numpy(), Unr)
    with pytest.raises(nm.NmError):
        nm.nm_admm_project(Wd, None, 128, 1024, 2, 4, 8, None)       # Z is required
    with pytest.raises(nm.NmError):
        nm.nm_admm_project(Wd, None, 128, 1022, 2, 4, 8, Z)          # in % m != 0
    with pytest.raises(nm.NmError):
        nm.nm_admm_project(Wd, None, 128, 1024, 3, 4, 8, Z)          # unsupported pattern
    # non-finite input raises the status bit
    Wbad = W.copy(); Wbad[5, 17] = np.inf
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_admm_project(to_dev(Wbad), None, 128, 1024, 2, 4, 8, Z, status=status)
    assert nm.nm_poll_status(status) == nm.NM_ERR_NONFINITE


def test_batched_admm_step_over_a_heterogeneous_layer():
    # the four matrices of a BERT-large layer, each with its own pattern and code width, in one call
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    cfgs = [(2, 4, 8), (1, 4, 4), (4, 8, 8), (4, 4, 4)]
    shapes = [(3072, 1024), (1024, 1024), (4096, 1024), (1024, 4096)]
    oracle.set_threads(oracle.max_threads())
    jobs, keep, refs = [], [], []
    for idx, ((out, k), (n, m, bits)) in enumerate(zip(shapes, cfgs)):
        W, U = wl.pack_sweep_matrix(3, 40 + idx, out, k)
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        Wd, Ud = to_dev(W), to_dev(U)
        Z = torch.full((out, k), float("nan"), dtype=torch.float32, device=DEV)
        Un = torch.full((out, k), float("nan"), dtype=torch.float32, device=DEV)
        v = torch.zeros(vb, dtype=torch.uint8, device=DEV)
        mt = torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV) if n != m else None
        sc = torch.zeros(out, dtype=torch.float32, device=DEV)
        # the third job asks for the dense outputs only
        jobs.append((Wd, Ud, n, m, bits, Z, Un, None if idx == 2 else v, None if idx == 2 else mt, None if idx == 2 else sc))
        keep.append((Z, Un, v, mt, sc))
        refs.append((oracle.admm_step(W, U, n, m, bits), oracle.project_pack(W, U, n, m, bits)))
    arr = nm.make_admm_jobs(jobs)
    ws_bytes = nm.nm_admm_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_admm_project_batched(arr, len(jobs), ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    for idx, ((Z, Un, v, mt, sc), ((Zr, Unr, sr), (vr, mr, s2))) in enumerate(zip(keep, refs)):
        assert np.array_equal(Z.cpu().numpy(), Zr) and np.array_equal(Un.cpu().numpy(), Unr), idx
        if idx != 2:
            assert np.array_equal(sc.cpu().numpy(), sr)
            assert np.array_equal(v.cpu().numpy(), np.asarray(vr).reshape(-1))
            if mt is not None:
                assert np.array_equal(mt.cpu().numpy().view(np.uint32), np.asarray(mr).reshape(-1))
    with pytest.raises(nm.NmError):
        nm.nm_admm_project_batched(arr, len(jobs), ws, ws_bytes - 1, status)   # workspace too small


@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 8, 8), (4, 8, 4), (4, 4, 8)])
@pytest.mark.parametrize("G", [1, 32, 64, 0, 100000])
def test_grouped_scales_pack_and_admm(n, m, bits, G):
    # several output channels per scale: packed outputs, Z and U_next against the oracle, bit for bit
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    oracle.set_threads(oracle.max_threads())
    for idx, (out, k) in enumerate([(300, 1024), (70, 4096), (45, 1032)]):
        if (k // m * n * bits) % 8:
            k *= 2
        W, U = wl.pack_sweep_matrix(3, 60 + idx, out, k)
        W[3] *= 20  # one channel far larger than the rest of its group
        vr, mr, sr = oracle.project_pack_grouped(W, U, n, m, bits, G)
        D = oracle.unpack(vr, mr, out, k, n, m, bits)
        Zr = (sr[:, None] * D.astype(np.float32)).astype(np.float32)
        Unr = ((W + U).astype(np.float32) - Zr).astype(np.float32)
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        Wd, Ud = to_dev(W), to_dev(U)
        v = torch.zeros(vb, dtype=torch.uint8, device=DEV)
        mt = torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV) if n != m else None
        sc = torch.full((out,), -1.0, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        nm.nm_project_pack_grouped(Wd, Ud, out, k, n, m, bits, G, v, mt, sc, status)
        assert nm.nm_poll_status(status) == nm.NM_OK
        assert np.array_equal(sc.cpu().numpy(), sr), (out, k)
        assert np.array_equal(v.cpu().numpy(), np.asarray(vr).reshape(-1))
        if mt is not None:
            assert np.array_equal(mt.cpu().numpy().view(np.uint32)[: mb // 4], np.asarray(mr).reshape(-1))
        Z = torch.empty((out, k), dtype=torch.float32, device=DEV)
        Un = torch.empty((out, k), dtype=torch.float32, device=DEV)
        sc2 = torch.zeros(out, dtype=torch.float32, device=DEV)
        nm.nm_admm_project_grouped(Wd, Ud, out, k, n, m, bits, G, Z, Un, None, None, sc2, status)
        assert nm.nm_poll_status(status) == nm.NM_OK
        assert np.array_equal(sc2.cpu().numpy(), sr)
        assert np.array_equal(Z.cpu().numpy(), Zr) and np.array_equal(Un.cpu().numpy(), Unr)


@pytest.mark.parametrize("G", [32, 0])
def test_grouped_scales_batched_over_a_heterogeneous_layer(G):
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    cfgs = [(2, 4, 8), (1, 4, 4), (4, 8, 8), (4, 4, 4), (2, 4, 8)]
    shapes = [(3072, 1024), (1000, 1024), (4096, 1024), (1024, 4096), (50, 8192)]
    oracle.set_threads(oracle.max_threads())
    jobs, keep, refs = [], [], []
    for idx, ((out, k), (n, m, bits)) in enumerate(zip(shapes, cfgs)):
        W, U = wl.pack_sweep_matrix(3, 80 + idx, out, k)
        W[out // 2] *= 30
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        v = torch.zeros(vb, dtype=torch.uint8, device=DEV)
        mt = torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV) if n != m else None
        sc = torch.full((out,), -3.0, dtype=torch.float32, device=DEV)
        jobs.append((to_dev(W), to_dev(U), n, m, bits, v, mt, sc))
        keep.append((v, mt, sc, mb))
        refs.append(oracle.project_pack_grouped(W, U, n, m, bits, G))
    arr = nm.make_pack_jobs(jobs)
    ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for _ in range(2):  # a second call must not see the first one's scales as maxima
        nm.nm_project_pack_grouped_batched(arr, len(jobs), G, ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    for idx, ((v, mt, sc, mb), (vr, mr, sr)) in enumerate(zip(keep, refs)):
        assert np.array_equal(sc.cpu().numpy(), sr), idx
        assert np.array_equal(v.cpu().numpy(), np.asarray(vr).reshape(-1)), idx
        if mt is not None:
            assert np.array_equal(mt.cpu().numpy().view(np.uint32)[: mb // 4], np.asarray(mr).reshape(-1)), idx


def test_grouped_admm_step_batched():
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    cfgs = [(2, 4, 8), (1, 4, 4), (4, 4, 8)]
    shapes = [(1000, 1024), (300, 4096), (2048, 1024)]
    G = 32
    oracle.set_threads(oracle.max_threads())
    jobs, keep, refs = [], [], []
    for idx, ((out, k), (n, m, bits)) in enumerate(zip(shapes, cfgs)):
        W, U = wl.pack_sweep_matrix(3, 90 + idx, out, k)
        W[7] *= 25
        Z = torch.empty((out, k), dtype=torch.float32, device=DEV)
        Un = torch.empty((out, k), dtype=torch.float32, device=DEV)
        sc = torch.zeros(out, dtype=torch.float32, device=DEV)
        jobs.append((to_dev(W), to_dev(U), n, m, bits, Z, Un, None, None, sc))
        keep.append((Z, Un, sc))
        vr, mr, sr = oracle.project_pack_grouped(W, U, n, m, bits, G)
        Zr = (sr[:, None] * oracle.unpack(vr, mr, out, k, n, m, bits).astype(np.float32)).astype(np.float32)
        refs.append((Zr, ((W + U).astype(np.float32) - Zr).astype(np.float32), sr))
    arr = nm.make_admm_jobs(jobs)
    ws_bytes = nm.nm_admm_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_admm_project_grouped_batched(arr, len(jobs), G, ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    for idx, ((Z, Un, sc), (Zr, Unr, sr)) in enumerate(zip(keep, refs)):
        assert np.array_equal(sc.cpu().numpy(), sr), idx
        assert np.array_equal(Z.cpu().numpy(), Zr) and np.array_equal(Un.cpu().numpy(), Unr), idx
