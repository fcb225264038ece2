"""GPU parity on seeded random shapes: token counts, reduction lengths, channel counts and patterns drawn so
that every kernel variant (CTA pairs with resident or streamed weights, one-CTA kernels with 192 / 128 / 64
token tiles, weight tiles built in shared memory per k-block or once per output tile) meets ragged token
and channel tails, single tiles and ranges that cross output tiles.  Accumulators bit for bit, fp32
outputs equal, int8 and bfloat16 outputs bit for bit (every third seed each)."""
import numpy as np
import pytest

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

MODES = [(2, 4, 8), (4, 4, 8), (2, 4, 4), (1, 4, 8), (1, 4, 4), (2, 8, 8), (2, 8, 4), (1, 8, 8), (1, 8, 4),
         (4, 4, 4), (4, 8, 8), (4, 8, 4)]


def _draw(rng):
    n, m, bits = MODES[int(rng.integers(0, len(MODES)))]
    K = 128 * int(rng.integers(1, 33))                                   # 128 .. 4096
    kind = int(rng.integers(0, 4))
    if kind == 0:      # small: a few tiles
        T, out = int(rng.integers(1, 400)), int(rng.integers(1, 400))
    elif kind == 1:    # tall: many token tiles, few channels
        T, out = int(rng.integers(2000, 20000)), int(rng.integers(1, 300))
    elif kind == 2:    # wide: many channels, few tokens
        T, out = int(rng.integers(1, 300)), int(rng.integers(500, 5000))
    else:              # enough tiles for every SM pair
        T, out = int(rng.integers(3000, 9000)), int(rng.integers(300, 1500))
    while T * K * out > 1.6e10:                                          # keep the oracle under a second
        if T > out:
            T = max(1, T // 2)
        else:
            out = max(1, out // 2)
    return T, K, out, n, m, bits


@pytest.mark.parametrize("seed", range(48))
def test_random_shape(seed):
    from gpu_util import PackedOnDevice, gpu_int_linear, gpu_int_linear_q8
    rng = np.random.default_rng(1000 + seed)
    T, K, out, n, m, bits = _draw(rng)
    W = wl.normal(rng, (out, K), 0.02)
    b = wl.normal(rng, (out,), 0.02)
    Xq = wl.random_int8([9, seed], (T, K))
    sx = np.float32(0.03)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    D = oracle.unpack(v, meta, out, K, n, m, bits)
    oracle.set_threads(oracle.max_threads())
    acc_ref, Y_ref = oracle.int_linear(Xq, D, sx, s, b)
    packed = PackedOnDevice(v, meta, s, out, K, n, m, bits)
    acc, Y = gpu_int_linear(Xq, packed, sx, b)
    tag = f"T={T} K={K} out={out} {n}:{m}/{bits}b"
    assert np.array_equal(acc, acc_ref), tag
    assert np.array_equal(Y, Y_ref), tag
    if seed % 3 == 0:
        sy = np.float32(max(np.abs(Y_ref).max(), 1e-3)) / np.float32(100.0)
        assert np.array_equal(gpu_int_linear_q8(Xq, packed, sx, b, sy), oracle.requantize_static(Y_ref, sy)), tag
    if seed % 3 == 1:
        from gpu_util import gpu_int_linear_bf16
        assert np.array_equal(gpu_int_linear_bf16(Xq, packed, sx, b), oracle.to_bf16(Y_ref)), tag


PACK_PATTERNS = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8), (4, 4)]


@pytest.mark.parametrize("seed", range(40))
def test_random_projection(seed):
    # projection / pack, the ADMM step and group-wise scales on random shapes: row lengths from one group to
    # several warps per row (not multiples of 1024), a handful to thousands of rows, with and without the dual
    import torch
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV
    rng = np.random.default_rng(2000 + seed)
    n, m = PACK_PATTERNS[int(rng.integers(0, len(PACK_PATTERNS)))]
    bits = int(rng.choice([8, 4]))
    k = 8 * int(rng.integers(1, 1300 if seed % 4 else 40))               # 8 .. 10392, multiples of 8
    while (k // m * n * bits) % 8:
        k += 8
    out = int(rng.integers(1, 3000 if k < 3000 else 300))
    G = int(rng.choice([1, 7, 32, 64, 0]))
    W = wl.tie_heavy(3000 + seed, out, k) if seed % 5 == 0 else wl.normal(rng, (out, k), 0.02)
    U = None if seed % 3 == 0 else wl.normal(rng, (out, k), 0.002)
    oracle.set_threads(oracle.max_threads())
    tag = f"out={out} in={k} {n}:{m}/{bits}b G={G}"
    vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
    Wd, Ud = to_dev(W), to_dev(U)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # ADMM step with every output
    Z = torch.empty((out, k), dtype=torch.float32, device=DEV)
    Un = torch.empty((out, k), dtype=torch.float32, device=DEV)
    v = torch.zeros(vb, dtype=torch.uint8, device=DEV)
    mt = torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=DEV) if n != m else None
    sc = torch.zeros(out, dtype=torch.float32, device=DEV)
    nm.nm_admm_project(Wd, Ud, out, k, n, m, bits, Z, Un, v, mt, sc, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    Zr, Unr, sr = oracle.admm_step(W, U, n, m, bits)
    vr, mr, _ = oracle.project_pack(W, U, n, m, bits)
    assert np.array_equal(Z.cpu().numpy(), Zr) and np.array_equal(Un.cpu().numpy(), Unr), tag
    assert np.array_equal(sc.cpu().numpy(), sr) and np.array_equal(v.cpu().numpy(), np.asarray(vr).reshape(-1)), tag
    if mt is not None:
        assert np.array_equal(mt.cpu().numpy().view(np.uint32)[: mb // 4], np.asarray(mr).reshape(-1)), tag
    # group-wise scales
    nm.nm_project_pack_grouped(Wd, Ud, out, k, n, m, bits, G, v, mt, sc, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    vg, mg, sg = oracle.project_pack_grouped(W, U, n, m, bits, G)
    assert np.array_equal(sc.cpu().numpy(), sg) and np.array_equal(v.cpu().numpy(), np.asarray(vg).reshape(-1)), tag
