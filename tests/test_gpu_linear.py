"""GPU parity: integer N:M linear layer against the CPU oracle.

int32 accumulators are compared bit for bit; fp32 outputs within 1e-5 relative / 1e-6 absolute
(and, since both sides round the same three operations, expected equal).
"""
import numpy as np
import pytest

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

MODES = [(2, 4, 8), (4, 4, 8)]  # weights already in the tensor core's form (TMA straight into the operand tile)
# weights rebuilt in shared memory: 4-bit codes, 1:4 / 2:8 / 1:8 into 2-of-4 slots, 4:8 and dense 4-bit into a dense tile
XFORM_MODES = [(2, 4, 4), (1, 4, 8), (1, 4, 4), (2, 8, 8), (2, 8, 4), (1, 8, 8), (1, 8, 4), (4, 4, 4), (4, 8, 8), (4, 8, 4)]
ALL_MODES = MODES + XFORM_MODES


def _case(seed, T, K, out, n, m, bits, tie=False):
    rng = np.random.default_rng(seed)
    W = wl.tie_heavy(seed, out, K) if tie else wl.normal(rng, (out, K), 0.02)
    b = wl.normal(rng, (out,), 0.02)
    X = wl.normal(rng, (T, K))
    Xq, sx = oracle.quantize_act(X)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    D = oracle.unpack(v, meta, out, K, n, m, bits)
    return Xq, sx, v, meta, s, b, D


def _run(seed, T, K, out, n, m, bits, tie=False, bias=True):
    from gpu_util import PackedOnDevice, gpu_int_linear, assert_close
    oracle.set_threads(oracle.max_threads())
    Xq, sx, v, meta, s, b, D = _case(seed, T, K, out, n, m, bits, tie)
    acc_ref, Y_ref = oracle.int_linear(Xq, D, sx, s, b if bias else None)
    packed = PackedOnDevice(v, meta, s, out, K, n, m, bits)
    acc, Y = gpu_int_linear(Xq, packed, sx, b if bias else None)
    assert np.array_equal(acc, acc_ref), f"{(acc != acc_ref).sum()} accumulators differ"
    assert_close(Y, Y_ref)
    assert np.array_equal(Y, Y_ref)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_single_tile(n, m, bits):
    _run(1, 64, 128, 128, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_one_tile_many_kblocks(n, m, bits):
    _run(2, 64, 1024, 128, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
@pytest.mark.parametrize("T", [1, 65, 129, 200])
def test_ragged_tokens(n, m, bits, T):
    _run(3 + T, T, 256, 256, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_ragged_out_and_no_bias(n, m, bits):
    _run(4, 100, 384, 200, n, m, bits, bias=False)
    _run(5, 70, 128, 8, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_bert_base_attention_projection(n, m, bits):
    # 128 tokens x 768 -> 768 (the small single-GEMM configuration)
    _run(0, 128, 768, 768, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_many_tiles_per_cta(n, m, bits):
    # enough tiles that every CTA walks several of them and changes output tile (192-token tiles)
    _run(6, 4096 + 37, 512, 1280, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
@pytest.mark.parametrize("T,K,out", [(8192 + 5, 1024, 1100), (6000, 384, 640), (6000, 128, 700)])
def test_short_reduction_many_token_tiles(n, m, bits, T, K, out):
    # reduction of at most eight k-blocks and several token tiles per CTA: in the transform modes the
    # weight tile is built once per output tile, kept in shared memory and rebuilt when a CTA moves on
    # to the next output tile (8, 3 and 1 k-blocks: more than, as many as, fewer than the builder groups)
    _run(8, T, K, out, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_longer_reduction_many_token_tiles(n, m, bits):
    # sixteen k-blocks: the transform modes build the weight tile of every k-block into the stage ring
    # (192-token tiles for the sparse targets), with a ragged last output tile and token tile
    _run(9, 6000 + 3, 2048, 600, n, m, bits)


@pytest.mark.parametrize("n,m,bits", ALL_MODES)
def test_tie_heavy_weights_and_extreme_activations(n, m, bits):
    from gpu_util import PackedOnDevice, gpu_int_linear
    _run(7, 150, 256, 128, n, m, bits, tie=True)
    # saturated operands: largest accumulator magnitudes
    K, out, T = 4096, 128, 64
    D = np.full((out, K), 127, np.int8) if n == m else None
    W = np.ones((out, K), np.float32)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    D = oracle.unpack(v, meta, out, K, n, m, bits)
    Xq = np.full((T, K), -128, np.int8)
    acc_ref, _ = oracle.int_linear(Xq, D, 1.0, s, None, want_y=False)
    acc, _ = gpu_int_linear(Xq, PackedOnDevice(v, meta, s, out, K, n, m, bits), 1.0, None)
    assert np.array_equal(acc, acc_ref)


def test_device_scale_and_running_absmax():
    import torch
    import paper_2206_15014_b200 as nm
    from gpu_util import PackedOnDevice, DEV, to_dev, assert_close
    Xq, sx, v, meta, s, b, D = _case(8, 300, 256, 384, 2, 4, 8)
    _, Y_ref = oracle.int_linear(Xq, D, sx, s, b)
    packed = PackedOnDevice(v, meta, s, 384, 256, 2, 4, 8)
    sxd = to_dev(np.array([sx], np.float32))
    amax = torch.zeros(1, dtype=torch.float32, device=DEV)
    Y = torch.empty((300, 384), dtype=torch.float32, device=DEV)
    nm.nm_int_linear_dsx(to_dev(Xq), 300, packed.desc, sxd, packed.scales, to_dev(b), Y, amax)
    assert nm.nm_poll_status() == 0
    assert_close(Y.cpu().numpy(), Y_ref)
    assert amax.item() == np.abs(Y_ref).max()


def test_linear_rejects_bad_arguments():
    import paper_2206_15014_b200 as nm
    assert nm.nm_int_linear_check(16, 128, 100, 2, 4, 8) == nm.NM_ERR_SHAPE
    assert nm.nm_int_linear_check(16, 128, 128, 3, 4, 8) == nm.NM_ERR_UNSUPPORTED
    assert nm.nm_int_linear_check(16, 128, 16384, 2, 4, 8) == nm.NM_ERR_UNSUPPORTED
    assert nm.nm_int_linear_check(16, 128, 128, 2, 4, 8) == nm.NM_OK


def test_linear_is_deterministic():
    from gpu_util import PackedOnDevice, gpu_int_linear
    Xq, sx, v, meta, s, b, D = _case(9, 500, 512, 256, 2, 4, 8)
    packed = PackedOnDevice(v, meta, s, 256, 512, 2, 4, 8)
    a = gpu_int_linear(Xq, packed, sx, b)
    c = gpu_int_linear(Xq, packed, sx, b)
    assert np.array_equal(a[0], c[0]) and np.array_equal(a[1], c[1])


@pytest.mark.parametrize("n,m,bits,K", [(2, 4, 8, 8192), (2, 4, 8, 6144), (4, 4, 8, 8192), (2, 4, 4, 6144), (1, 8, 8, 8192)])
def test_long_reductions(n, m, bits, K):
    # reductions beyond 4096: the metadata of one output tile only fits next to 128-token accumulators
    _run(10 + K, 300, K, 256, n, m, bits)


def test_largest_accumulators_fit_int32():
    # K = 8192 with saturated operands: |acc| = 8192 * 128 * 127 < 2^31
    from gpu_util import PackedOnDevice, gpu_int_linear
    K, out, T = 8192, 128, 40
    W = np.ones((out, K), np.float32)
    v, meta, s = oracle.project_pack(W, None, 4, 4, 8)
    D = oracle.unpack(v, meta, out, K, 4, 4, 8)
    Xq = np.full((T, K), -128, np.int8)
    acc_ref, _ = oracle.int_linear(Xq, D, 1.0, s, None, want_y=False)
    acc, _ = gpu_int_linear(Xq, PackedOnDevice(v, meta, s, out, K, 4, 4, 8), 1.0, None)
    assert np.array_equal(acc, acc_ref) and acc.min() == -8192 * 128 * 127


def test_linear_argument_errors():
    import torch
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV
    X = torch.zeros((16, 128), dtype=torch.int8, device=DEV)
    vals = torch.zeros(128 * 64 + 16, dtype=torch.uint8, device=DEV)
    meta = torch.zeros(128 * 4, dtype=torch.int32, device=DEV)
    sw = torch.ones(128, device=DEV)
    Y = torch.zeros((16, 128), device=DEV)
    good = nm.make_packed(128, 128, 2, 4, 8, vals, meta)
    nm.nm_int_linear(X, 16, good, 1.0, sw, None, Y)
    for call, code in [
        (lambda: nm.nm_int_linear(None, 16, good, 1.0, sw, None, Y), nm.NM_ERR_NULL),
        (lambda: nm.nm_int_linear(X, 16, good, 1.0, None, None, Y), nm.NM_ERR_NULL),
        (lambda: nm.nm_int_linear(X, 16, nm.make_packed(128, 128, 2, 4, 8, vals, None), 1.0, sw, None, Y), nm.NM_ERR_NULL),
        (lambda: nm.nm_int_linear(X.view(-1)[1:], 15, good, 1.0, sw, None, Y), nm.NM_ERR_ALIGN),
        (lambda: nm.nm_int_linear(X, 16, nm.make_packed(128, 128, 2, 4, 8, vals[1:], meta), 1.0, sw, None, Y), nm.NM_ERR_ALIGN),
        (lambda: nm.nm_int_linear(X, 16, nm.make_packed(128, 96, 2, 4, 8, vals, meta), 1.0, sw, None, Y), nm.NM_ERR_SHAPE),
        (lambda: nm.nm_int_linear(X, -1, good, 1.0, sw, None, Y), nm.NM_ERR_SHAPE),
        (lambda: nm.nm_int_linear(X, 16, nm.make_packed(128, 128, 2, 4, 6, vals, meta), 1.0, sw, None, Y), nm.NM_ERR_UNSUPPORTED),
    ]:
        with pytest.raises(nm.NmError) as e:
            call()
        assert e.value.code == code
    nm.nm_int_linear(X, 0, good, 1.0, sw, None, Y)  # no tokens: nothing to do
    assert nm.nm_poll_status() == nm.NM_OK
