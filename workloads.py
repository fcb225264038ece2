"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds no arithmetic of the method (no projection, no quantiser, no
GEMM): it only draws random tensors with the shapes and value distributions of
BERT-base / BERT-large encoder linears and of the batch x sequence grid of the
paper's inference table (Table 3: sequence 128 / 384, batch up to 128).  They
stand in for fine-tuned weights and real activations.

Generator: numpy PCG64 (``numpy.random.default_rng(seed)``), ``standard_normal``
in float32, drawn in the order documented per function, scaled in float32.
"""
from __future__ import annotations

import numpy as np

# (name, in features K, out features) of the four GEMMs of one encoder layer.
BERT_BASE_GEMMS = (("qkv", 768, 2304), ("attn_out", 768, 768), ("ffn1", 768, 3072), ("ffn2", 3072, 768))
BERT_LARGE_GEMMS = (("qkv", 1024, 3072), ("attn_out", 1024, 1024), ("ffn1", 1024, 4096), ("ffn2", 4096, 1024))

# (n kept, m group, bits) variants of the projection/pack sweep.
PACK_SWEEP = tuple((n, m, b) for (n, m) in ((1, 4), (2, 4), (2, 8), (4, 8)) for b in (8, 4))

# Modes of the heterogeneous chain: (n, m, bits); dense int8 is (4, 4, 8).
CHAIN_MODES = ((4, 4, 8), (2, 4, 8), (2, 4, 4), (1, 4, 8), (4, 8, 8))

W_STD = np.float32(0.02)
U_STD = np.float32(0.002)


def normal(rng, shape, std=1.0):
    return rng.standard_normal(shape, dtype=np.float32) * np.float32(std)


def linear_case(seed, tokens, k, out):
    """One GEMM: draws X[tokens,k] ~ N(0,1), W[out,k] ~ N(0,0.02), b[out] ~ N(0,0.02)."""
    rng = np.random.default_rng(seed)
    X = normal(rng, (tokens, k))
    W = normal(rng, (out, k), W_STD)
    b = normal(rng, (out,), W_STD)
    return X, W, b


def single_projection_case(seed=0):
    """BERT-base attention output projection at 128 tokens (hidden 768)."""
    return linear_case(seed, 128, 768, 768)


def encoder_layer_cases(seed, tokens, gemms):
    """For each GEMM of one encoder layer, in order: X[tokens,K], W[out,K], b[out]."""
    rng = np.random.default_rng(seed)
    cases = []
    for name, k, out in gemms:
        X = normal(rng, (tokens, k))
        W = normal(rng, (out, k), W_STD)
        b = normal(rng, (out,), W_STD)
        cases.append((name, X, W, b))
    return cases


def pack_sweep_shapes(layers=24, gemms=BERT_LARGE_GEMMS):
    """[(out, in)] of every encoder linear weight, layer by layer (fused QKV counts once)."""
    return [(out, k) for _ in range(layers) for (_, k, out) in gemms]


def pack_sweep_matrix(seed, index, out, k):
    """Weight W ~ N(0,0.02) and ADMM dual U ~ N(0,0.002) of matrix `index` of the sweep."""
    rng = np.random.default_rng([seed, index])
    W = normal(rng, (out, k), W_STD)
    U = normal(rng, (out, k), U_STD)
    return W, U


def chain_case(seed=4, layers=12, tokens=6144, gemms=BERT_BASE_GEMMS):
    """Heterogeneous encoder GEMM chain: modes[layers,4] in 0..4, h0[tokens,hidden], then per
    layer and GEMM W ~ N(0,0.02), b ~ N(0,0.02)."""
    rng = np.random.default_rng(seed)
    modes = rng.integers(0, len(CHAIN_MODES), size=(layers, len(gemms)))
    h0 = normal(rng, (tokens, gemms[0][1]))
    weights = []
    for _ in range(layers):
        layer = []
        for _, k, out in gemms:
            layer.append((normal(rng, (out, k), W_STD), normal(rng, (out,), W_STD)))
        weights.append(layer)
    return modes, h0, weights


def tie_heavy(seed, out, k, levels=5):
    """Weights on a coarse grid (small integers x 2^-7): many equal magnitudes, +-pairs, zeros."""
    rng = np.random.default_rng(seed)
    return (rng.integers(-levels, levels + 1, size=(out, k)).astype(np.float32)
            * np.float32(2.0 ** -7))


def with_outliers(seed, out, k, per_row=3, sigma=10.0):
    """N(0,0.02) weights with a few 10-sigma outliers per row, one all-zero row and zero groups."""
    rng = np.random.default_rng(seed)
    W = normal(rng, (out, k), W_STD)
    cols = rng.integers(0, k, size=(out, per_row))
    sign = rng.integers(0, 2, size=(out, per_row)).astype(np.float32) * 2 - 1
    for r in range(out):
        W[r, cols[r]] = sign[r] * np.float32(sigma) * W_STD
    if out > 2:
        W[out // 2, :] = 0.0
    W[0, : min(k, 16)] = 0.0
    return W


def random_int8(seed, shape):
    rng = np.random.default_rng(seed)
    return rng.integers(-128, 128, size=shape, dtype=np.int8)
