"""GPU parity on seeded random shapes: token counts, reduction lengths, channel counts and patterns drawn so
that every kernel variant (CTA pairs with resident or streamed weights, one-CTA kernels with 192 / 128 / 64
token tiles, weight tiles built in shared memory per k-block or once per output tile) meets ragged token
and channel tails, single tiles and ranges that cross output tiles.  Accumulators bit for bit, fp32
outputs equal, int8 outputs bit for bit."""
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
