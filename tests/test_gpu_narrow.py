"""GPU parity: int8 (static scale, Eq. 5 with b = 8) and bfloat16 outputs of the N:M integer linear layer.

Both sides form y with the same three fp32 operations (int -> float, one multiply for sx * sw[o], one
fma with the bias), divide by the scale with an IEEE division and round half to even, so the int8 codes
and the bfloat16 bit patterns are compared bit for bit.
"""
import numpy as np
import pytest

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

# int8 2:4 and dense (TMA weights, CTA pairs when large), and weights rebuilt in shared memory
MODES = [(2, 4, 8), (4, 4, 8), (2, 4, 4), (1, 4, 8), (2, 8, 8), (4, 8, 8)]
# (tokens, K, out): one tile; ragged, out % 16 != 0 (plain stores) ; out % 16 == 0 but ragged tokens;
# many tiles with resident weights and output-tile changes; long reduction with streamed weights
# the last one: resident weights on CTA pairs with rows that no TMA store can address (plain stores from sixteen warps)
SHAPES = [(64, 128, 128), (100, 384, 200), (77, 256, 208), (4096 + 37, 512, 1280), (6000 + 3, 2048, 640), (7680 + 5, 512, 516)]


def _setup(seed, T, K, out, n, m, bits):
    rng = np.random.default_rng(seed)
    W = wl.normal(rng, (out, K), 0.02)
    b = wl.normal(rng, (out,), 0.02)
    X = wl.normal(rng, (T, K))
    Xq, sx = oracle.quantize_act(X)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    D = oracle.unpack(v, meta, out, K, n, m, bits)
    oracle.set_threads(oracle.max_threads())
    _, Y = oracle.int_linear(Xq, D, sx, s, b, want_acc=False)
    return Xq, sx, v, meta, s, b, Y


@pytest.mark.parametrize("n,m,bits", MODES)
@pytest.mark.parametrize("T,K,out", SHAPES)
def test_int8_output_matches_oracle(n, m, bits, T, K, out):
    from gpu_util import PackedOnDevice, gpu_int_linear_q8
    Xq, sx, v, meta, s, b, Y = _setup(21, T, K, out, n, m, bits)
    packed = PackedOnDevice(v, meta, s, out, K, n, m, bits)
    amax = np.float32(np.abs(Y).max())
    for sy in (amax / np.float32(127.0), amax / np.float32(40.0)):  # full range; two thirds of the outputs clamp
        ref = oracle.requantize_static(Y, sy)
        got = gpu_int_linear_q8(Xq, packed, sx, b, sy)
        assert np.array_equal(got, ref), f"{(got != ref).sum()} of {ref.size} codes differ at sy={sy}"


@pytest.mark.parametrize("n,m,bits", MODES)
@pytest.mark.parametrize("T,K,out", SHAPES)
def test_bf16_output_matches_oracle(n, m, bits, T, K, out):
    from gpu_util import PackedOnDevice, gpu_int_linear_bf16
    Xq, sx, v, meta, s, b, Y = _setup(22, T, K, out, n, m, bits)
    got = gpu_int_linear_bf16(Xq, PackedOnDevice(v, meta, s, out, K, n, m, bits), sx, b)
    ref = oracle.to_bf16(Y)
    assert np.array_equal(got, ref), f"{(got != ref).sum()} of {ref.size} patterns differ"


def test_int8_chain_of_two_layers():
    # layer 1 writes int8 with a static scale; layer 2 consumes it as its X with sx = that scale
    from gpu_util import PackedOnDevice, gpu_int_linear, gpu_int_linear_q8
    T, K, H, out = 1000, 768, 3072, 768
    rng = np.random.default_rng(23)
    W1, b1 = wl.normal(rng, (H, K), 0.02), wl.normal(rng, (H,), 0.02)
    W2, b2 = wl.normal(rng, (out, H), 0.02), wl.normal(rng, (out,), 0.02)
    Xq, sx = oracle.quantize_act(wl.normal(rng, (T, K)))
    v1, m1, s1 = oracle.project_pack(W1, None, 2, 4, 8)
    v2, m2, s2 = oracle.project_pack(W2, None, 2, 4, 4)
    oracle.set_threads(oracle.max_threads())
    _, Y1 = oracle.int_linear(Xq, oracle.unpack(v1, m1, H, K, 2, 4, 8), sx, s1, b1, want_acc=False)
    sy = np.float32(np.abs(Y1).max()) / np.float32(127.0)
    H1 = oracle.requantize_static(Y1, sy)
    acc2, Y2 = oracle.int_linear(H1, oracle.unpack(v2, m2, out, H, 2, 4, 4), sy, s2, b2)
    g1 = gpu_int_linear_q8(Xq, PackedOnDevice(v1, m1, s1, H, K, 2, 4, 8), sx, b1, sy)
    assert np.array_equal(g1, H1)
    gacc2, gY2 = gpu_int_linear(g1, PackedOnDevice(v2, m2, s2, out, H, 2, 4, 4), sy, b2)
    assert np.array_equal(gacc2, acc2) and np.array_equal(gY2, Y2)


@pytest.mark.parametrize("T,K,out", [(300, 4096, 128), (8960, 1024, 512), (8960, 4096, 512)])
@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (4, 4, 8), (2, 4, 4)])
def test_accumulators_from_zero_to_the_largest(n, m, bits, T, K, out):
    """Constant rows of X against all-ones weights give every token its own accumulator value, from 0 up to the
    largest the operands allow (beyond 2^22 and 2^24 in magnitude for 8-bit codes, where int -> float rounds): fp32,
    int8 and bfloat16 outputs bit for bit on the one-CTA, resident-weight pair and 512-channel pair kernels."""
    from gpu_util import PackedOnDevice, gpu_int_linear, gpu_int_linear_q8, gpu_int_linear_bf16
    oracle.set_threads(oracle.max_threads())
    W = np.ones((out, K), np.float32)
    b = wl.normal(np.random.default_rng(31), (out,), 0.5)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    D = oracle.unpack(v, meta, out, K, n, m, bits)
    c = ((np.arange(T) * 37) % 256 - 128).astype(np.int8)
    Xq = np.repeat(c[:, None], K, axis=1)
    sx = np.float32(2e-4)
    acc_ref, Y = oracle.int_linear(Xq, D, sx, s, b)
    if bits == 8:
        assert np.abs(acc_ref).max() > (1 << 22)
    packed = PackedOnDevice(v, meta, s, out, K, n, m, bits)
    acc, Yg = gpu_int_linear(Xq, packed, sx, b)
    assert np.array_equal(acc, acc_ref) and np.array_equal(Yg, Y)
    sy = np.float32(np.abs(Y).max()) / np.float32(127.0)
    assert np.array_equal(gpu_int_linear_q8(Xq, packed, sx, b, sy), oracle.requantize_static(Y, sy))
    assert np.array_equal(gpu_int_linear_bf16(Xq, packed, sx, b), oracle.to_bf16(Y))


def test_narrow_outputs_reject_bad_arguments():
    import torch
    import paper_2206_15014_b200 as nm
    from gpu_util import PackedOnDevice, to_dev
    rng = np.random.default_rng(24)
    v, meta, s = oracle.project_pack(wl.normal(rng, (128, 128), 0.02), None, 2, 4, 8)
    packed = PackedOnDevice(v, meta, s, 128, 128, 2, 4, 8)
    X = to_dev(np.zeros((16, 128), np.int8))
    Yq = torch.zeros((16, 128), dtype=torch.int8, device="cuda")
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(nm.NmError):
            nm.nm_int_linear_q8(X, 16, packed.desc, 1.0, packed.scales, None, bad, Yq)
    with pytest.raises(nm.NmError):
        nm.nm_int_linear_q8(X, 16, packed.desc, 1.0, packed.scales, None, 1.0, None)
    with pytest.raises(nm.NmError):
        nm.nm_int_linear_bf16(X, 16, packed.desc, 1.0, None, None, Yq)
    with pytest.raises(nm.NmError):  # bfloat16 output on an odd byte address
        buf = torch.zeros(16 * 128 * 2 + 2, dtype=torch.uint8, device="cuda")
        nm.nm_int_linear_bf16(X, 16, packed.desc, 1.0, packed.scales, None, buf[1:], None)
