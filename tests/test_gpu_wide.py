"""GPU parity of the 512-channel CTA-pair kernel (2:4 weights with 8-bit codes, or packed 4-bit codes widened in shared
memory by its builder warps; reduction longer than 1024) against the CPU oracle.

The library picks that kernel only for problems with at least one tile per SM pair; the option "wide_any"
sends every eligible shape to it, so that small and ragged cases (one tile, a ragged last token tile, an output
that does not fill the second block of 128 channels, few and many pipeline stages per tile, a pair that walks
several tiles and changes output tile) reach it too.  int32 accumulators bit for bit, fp32 outputs equal, and the
kernel's int8 and bfloat16 outputs bit for bit.
"""
import numpy as np
import pytest

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=[224, 192])
def wide_kernel_everywhere(request):
    """Every test runs with both token-tile widths of the kernel."""
    import paper_2206_15014_b200 as nm
    nm.nm_debug_set_option("wide_any", 1)
    nm.nm_debug_set_option("wide_bn", request.param)
    yield request.param
    nm.nm_debug_set_option("wide_any", 0)
    nm.nm_debug_set_option("wide_bn", 0)


def _run(seed, T, K, out, tie=False, bias=True, bits=8, narrow=True):
    from gpu_util import PackedOnDevice, gpu_int_linear, assert_close
    oracle.set_threads(oracle.max_threads())
    rng = np.random.default_rng(seed)
    W = wl.tie_heavy(seed, out, K) if tie else wl.normal(rng, (out, K), 0.02)
    b = wl.normal(rng, (out,), 0.02)
    Xq, sx = oracle.quantize_act(wl.normal(rng, (T, K)))
    v, meta, s = oracle.project_pack(W, None, 2, 4, bits)
    D = oracle.unpack(v, meta, out, K, 2, 4, bits)
    acc_ref, Y_ref = oracle.int_linear(Xq, D, sx, s, b if bias else None)
    packed = PackedOnDevice(v, meta, s, out, K, 2, 4, bits)
    acc, Y = gpu_int_linear(Xq, packed, sx, b if bias else None)
    assert np.array_equal(acc, acc_ref), f"{(acc != acc_ref).sum()} accumulators differ"
    assert_close(Y, Y_ref)
    assert np.array_equal(Y, Y_ref)
    if narrow:   # the same kernel's int8 (two scales: full range; two thirds of the outputs clamp) and bfloat16 outputs
        from gpu_util import gpu_int_linear_q8, gpu_int_linear_bf16
        amax = np.float32(np.abs(Y_ref).max())
        for sy in (amax / np.float32(127.0), amax / np.float32(40.0)):
            ref = oracle.requantize_static(Y_ref, sy)
            got = gpu_int_linear_q8(Xq, packed, sx, b if bias else None, sy)
            assert np.array_equal(got, ref), f"{(got != ref).sum()} of {ref.size} codes differ at sy={sy}"
        got = gpu_int_linear_bf16(Xq, packed, sx, b if bias else None)
        assert np.array_equal(got, oracle.to_bf16(Y_ref)), "bfloat16 patterns differ"


@pytest.mark.parametrize("T,K,out", [
    (224, 1152, 512),      # one full tile, nine stages (more than the ring holds)
    (100, 1152, 300),      # one ragged tile: second block partly filled, 100 of 224 tokens
    (1, 1280, 257),        # a single token; one channel in the second block
    (225, 2048, 513),      # two token tiles x two output tiles, the second ones almost empty
    (448, 1536, 1024),     # four tiles
    (700, 8192, 520),      # longest supported reduction (64 stages per tile)
])
@pytest.mark.parametrize("bits", [8, 4])
def test_small_and_ragged(T, K, out, bits):
    _run(11 + T, T, K, out, bits=bits)


@pytest.mark.parametrize("bits", [8, 4])
def test_no_bias_and_ties(bits):
    _run(21, 300, 1152, 640, tie=True, bias=False, bits=bits)


def test_many_tiles_per_pair():
    # 5 output tiles x 34 token tiles = 170 tiles on 74 pairs: every pair walks two or three tiles, most change
    # output tile inside their range; the last token tile is ragged
    _run(22, 34 * 224 - 77, 1152, 2400)


def test_many_tiles_per_pair_packed_4_bit():
    _run(25, 34 * 224 - 77, 1152, 2400, bits=4)


def test_library_choice_of_tile_width():
    # no forced width: 12288 tokens x 1536 channels gives the slowest pair less to do with 192-token tiles
    import paper_2206_15014_b200 as nm
    nm.nm_debug_set_option("wide_bn", 0)
    nm.nm_debug_set_option("wide_any", 0)
    _run(23, 12288, 1280, 1536)


def test_output_rows_not_16_byte_aligned():
    # out % 4 != 0: the epilogue stores directly instead of through TMA
    _run(24, 500, 1152, 515)
    _run(26, 500, 1152, 515, bits=4)
