"""CPU checks that pin the oracle to what the paper and the mathematics fix.

Each test names the passage it follows.  None of them calls the CUDA library.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
import workloads as wl

PATTERNS = [(1, 4), (2, 4), (1, 8), (2, 8), (4, 8)]
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_tables.txt")


def _fields(meta_row, count, fb):
    """Decode `count` fb-bit fields, LSB first, from little-endian u32 words."""
    out = []
    for e in range(count):
        bit = e * fb
        out.append(int((int(meta_row[bit // 32]) >> (bit % 32)) & ((1 << fb) - 1)))
    return out


def _codes(values_row, count, bits):
    if bits == 8:
        return [int(np.int8(values_row[e])) for e in range(count)]
    out = []
    for e in range(count):
        nib = (int(values_row[e // 2]) >> (4 if e & 1 else 0)) & 0xF
        out.append(nib - 16 if nib >= 8 else nib)
    return out


# ----------------------------------------------------------------------------------------------
# Hand-worked example of the documented packing (2:4, 8 bit and 4 bit).
# ----------------------------------------------------------------------------------------------
def test_hand_worked_pack_example():
    # Row of 8 = two groups of 4.  max|v| = 1.0 -> s8 = 1/127, s4 = 1/7.
    # Group 0: |.5| = |-.5| = |.5| tie -> the two lowest indices 0,1 are kept.
    # Group 1: 1.0 (pos 0) and 0.3 (pos 3) are the two largest magnitudes.
    W = np.array([[0.5, -0.5, 0.5, 0.25, 1.0, 0.1, -0.2, 0.3]], dtype=np.float32)
    v, m, s = oracle.project_pack(W, None, 2, 4, 8)
    assert s[0] == np.float32(1.0) / np.float32(127.0)
    # 0.5*127 = 63.5 -> half to even -> 64; 0.3*127 = 38.1 -> 38
    assert v.tolist() == [[64, 256 - 64, 127, 38]]
    # fields (LSB first, 2 bits each): 0,1 | 0,3 -> 0b11_00_01_00 = 0xC4
    assert m.tolist() == [[0xC4]]
    v4, m4, s4 = oracle.project_pack(W, None, 2, 4, 4)
    assert s4[0] == np.float32(1.0) / np.float32(7.0)
    # fl32(1/7) lies just above 1/7, so 0.5 / s = 3.4999998 (a true division, not 0.5 * 7) -> 3;
    # codes 3, -3, 7, 2.1 -> 2 ; nibbles 3, 0xD, 7, 2 ; even element in the low nibble
    assert v4.tolist() == [[0xD3, 0x27]]
    assert m4.tolist() == [[0xC4]]
    assert oracle.unpack(v4, m4, 1, 8, 2, 4, 4).tolist() == [[3, -3, 0, 0, 7, 0, 0, 2]]


def test_hand_worked_m8_example():
    # One group of 8, keep 2: magnitudes 9 (pos 6) and 8 (pos 1); 4-bit fields.
    W = np.array([[1, -8, 2, 3, 0, 4, 9, -5]], dtype=np.float32)
    v, m, s = oracle.project_pack(W, None, 2, 8, 8)
    assert s[0] == np.float32(9.0) / np.float32(127.0)
    assert _codes(v[0], 2, 8) == [int(np.rint(np.float32(-8) / s[0])), 127]
    assert m.tolist() == [[0x61]]  # fields 1 then 6
    # keep 4 of 8: positions of 9, 8, 5, 4 -> ascending 1,5,6,7
    v, m, s = oracle.project_pack(W, None, 4, 8, 8)
    assert m.tolist() == [[0x7651]]


# ----------------------------------------------------------------------------------------------
# T1: structure of the packed form (Sec. 1: at most n non-zeros per group of m)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_structure(n, m, bits):
    W = wl.normal(np.random.default_rng(10), (24, 64), 0.02)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    fb = 2 if m == 4 else 4
    D = oracle.unpack(v, meta, 24, 64, n, m, bits)
    for r in range(24):
        f = _fields(meta[r], 64 // m * n, fb)
        for g in range(64 // m):
            pos = f[g * n:(g + 1) * n]
            assert all(p < m for p in pos)
            assert all(a < b for a, b in zip(pos, pos[1:]))
        assert (np.count_nonzero(D[r].reshape(-1, m), axis=1) <= n).all()


# ----------------------------------------------------------------------------------------------
# T2: the support is the Euclidean projection's (Eq. 2-3), brute force over all C(m,n) supports
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,m", PATTERNS + [(3, 4), (5, 8)])
def test_projection_is_euclidean_bruteforce(n, m):
    rng = np.random.default_rng(20 + n * 10 + m)
    rows = [wl.normal(rng, (m,), 0.02) for _ in range(40)]
    rows += [rng.integers(-2, 3, size=m).astype(np.float32) for _ in range(120)]  # tie-heavy
    rows += [np.zeros(m, np.float32), np.ones(m, np.float32), -np.ones(m, np.float32)]
    for v in rows:
        Z = oracle.project_dense(v[None, :], None, n, m)[0]
        got = None
        best, best_sup = None, None
        for sup in itertools.combinations(range(m), n):
            d = sum(Fraction(float(v[i])) ** 2 for i in range(m) if i not in sup)
            if best is None or d < best:  # strict: first (lexicographically smallest) minimiser wins
                best, best_sup = d, sup
        # distance attained by the oracle's Z
        d_or = sum((Fraction(float(v[i])) - Fraction(float(Z[i]))) ** 2 for i in range(m))
        assert d_or == best
        # kept entries are unchanged, and the support is the lexicographically smallest minimiser
        expect = np.zeros(m, np.float32)
        expect[list(best_sup)] = v[list(best_sup)]
        assert np.array_equal(Z, expect), (v, Z, best_sup, got)


def test_projection_support_matches_pack_metadata():
    W = wl.tie_heavy(21, 16, 64)
    for n, m in PATTERNS:
        Z = oracle.project_dense(W, None, n, m)
        v, meta, s = oracle.project_pack(W, None, n, m, 8)
        fb = 2 if m == 4 else 4
        for r in range(16):
            f = _fields(meta[r], 64 // m * n, fb)
            mask = np.zeros(64, bool)
            for g in range(64 // m):
                for p in f[g * n:(g + 1) * n]:
                    mask[g * m + p] = True
            assert np.array_equal(np.where(mask, W[r], 0), Z[r])


# ----------------------------------------------------------------------------------------------
# T3: idempotence of the projection (Sec. 3.2) and of the joint operator
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,m", PATTERNS)
def test_idempotence(n, m):
    for W in (wl.normal(np.random.default_rng(30), (12, 96), 0.02), wl.tie_heavy(31, 12, 96)):
        Z = oracle.project_dense(W, None, n, m)
        assert np.array_equal(oracle.project_dense(Z, None, n, m), Z)
        for bits in (8, 4):
            v, meta, s = oracle.project_pack(W, None, n, m, bits)
            D = oracle.unpack(v, meta, 12, 96, n, m, bits)
            Zq = s[:, None] * D.astype(np.float32)
            v2, meta2, s2 = oracle.project_pack(Zq, None, n, m, bits)
            D2 = oracle.unpack(v2, meta2, 12, 96, n, m, bits)
            assert np.array_equal(D, D2)
            assert np.allclose(s, s2, rtol=2e-7, atol=0)


# ----------------------------------------------------------------------------------------------
# T4: ADMM-Max scale is unchanged by pruning first (Sec. 3.3.1, last paragraph)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,m", PATTERNS)
def test_scale_order_invariance(n, m):
    for W in (wl.normal(np.random.default_rng(40), (32, 128), 0.02), wl.tie_heavy(41, 32, 128),
              wl.with_outliers(42, 32, 128)):
        U = wl.normal(np.random.default_rng(43), W.shape, 0.002)
        for bits in (8, 4):
            s_joint = oracle.project_pack(W, U, n, m, bits)[2]
            s_pruned = oracle.row_scales(oracle.project_dense(W, U, n, m), bits)
            s_raw = oracle.row_scales(W + U, bits)
            assert np.array_equal(s_joint, s_pruned)
            assert np.array_equal(s_joint, s_raw)


# ----------------------------------------------------------------------------------------------
# T5: quantiser range (Eq. 5) under the ADMM-Max scale
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [8, 4])
def test_quantiser_range_and_error(bits):
    qmax = 2 ** (bits - 1) - 1
    W = wl.with_outliers(50, 48, 256)
    U = wl.normal(np.random.default_rng(51), W.shape, 0.002)
    V = W + U
    for n, m in PATTERNS:
        v, meta, s = oracle.project_pack(W, U, n, m, bits)
        D = oracle.unpack(v, meta, 48, 256, n, m, bits).astype(np.int32)
        assert D.min() >= -qmax  # -2^(b-1) is unreachable with s = max|v| / qmax
        assert D.max() <= qmax
        Z = oracle.project_dense(W, U, n, m)
        kept = Z != 0
        err = np.abs(Z.astype(np.float64) - s[:, None].astype(np.float64) * D)
        bound = s[:, None].astype(np.float64) * 0.5 * (1 + 2 ** -20)
        assert (err[kept] <= np.broadcast_to(bound, err.shape)[kept]).all()
        for r in range(48):
            a = np.abs(V[r]).max()
            if a == 0:
                assert s[r] == 1 and not D[r].any()
            else:
                k = int(np.abs(V[r]).argmax())
                assert abs(D[r, k]) == qmax


# ----------------------------------------------------------------------------------------------
# T6: dequant(quant) == STE fake-quant forward (Sec. 3.3.2, Eq. 4)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,m", PATTERNS)
@pytest.mark.parametrize("bits", [8, 4])
def test_dequant_equals_fake_quant(n, m, bits):
    W = wl.normal(np.random.default_rng(60), (16, 64), 0.02)
    U = wl.normal(np.random.default_rng(61), (16, 64), 0.002)
    v, meta, s = oracle.project_pack(W, U, n, m, bits)
    D = oracle.unpack(v, meta, 16, 64, n, m, bits)
    deq = s[:, None] * D.astype(np.float32)
    fq = oracle.fake_quant(oracle.project_dense(W, U, n, m), bits, s)
    assert np.array_equal(deq, fq)


# ----------------------------------------------------------------------------------------------
# T7: n == m is textbook per-channel absmax quantisation (Sec. 1: symmetric scalar quantiser)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [8, 4])
def test_dense_reduces_to_absmax_quantisation(bits):
    W = wl.with_outliers(70, 20, 96)
    qmax = 2 ** (bits - 1) - 1
    v, meta, s = oracle.project_pack(W, None, 4, 4, bits)
    D = oracle.unpack(v, None, 20, 96, 4, 4, bits)
    amax = np.abs(W).max(axis=1)
    s_ref = np.where(amax == 0, np.float32(1), amax / np.float32(qmax)).astype(np.float32)
    D_ref = np.clip(np.rint(W / s_ref[:, None]), -qmax - 1, qmax).astype(np.int8)
    assert np.array_equal(s, s_ref)
    assert np.array_equal(D, D_ref)
    assert meta.size == 0


# ----------------------------------------------------------------------------------------------
# T8 / T9: integer GEMM against numpy int64 matmul; skipping pruned positions changes nothing
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T", [1, 5, 33])
@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 4, 8), (4, 8, 8), (2, 8, 4), (4, 4, 8)])
def test_int_linear_matches_numpy(T, n, m, bits):
    K, out = 64, 24
    X = wl.random_int8(80 + T, (T, K))
    W = wl.normal(np.random.default_rng(81), (out, K), 0.02)
    v, meta, s = oracle.project_pack(W, None, n, m, bits)
    D = oracle.unpack(v, meta, out, K, n, m, bits)
    acc, _ = oracle.int_linear(X, D, 1.0, s, None, want_y=False)
    ref = X.astype(np.int64) @ D.astype(np.int64).T
    assert np.array_equal(acc.astype(np.int64), ref)
    assert np.array_equal(oracle.int_linear_kept(X, v, meta, out, K, n, m, bits), acc)


def test_int_linear_extremes_and_single_group():
    X = np.full((3, 4), -128, np.int8)
    D = np.full((2, 4), -128, np.int8)
    acc, _ = oracle.int_linear(X, D, 1.0, np.ones(2, np.float32), None, want_y=False)
    assert (acc == 4 * 128 * 128).all()
    X = np.full((2, 4096), 127, np.int8)
    D = np.full((1, 4096), -127, np.int8)
    acc, _ = oracle.int_linear(X, D, 1.0, np.ones(1, np.float32), None, want_y=False)
    assert (acc == -4096 * 127 * 127).all()


# ----------------------------------------------------------------------------------------------
# T10: fp32 epilogue (Eq. 4) against the same expression in double
# ----------------------------------------------------------------------------------------------
def test_epilogue_against_double():
    T, K, out = 17, 128, 40
    X = wl.random_int8(90, (T, K))
    W = wl.normal(np.random.default_rng(91), (out, K), 0.02)
    b = wl.normal(np.random.default_rng(92), (out,), 0.02)
    v, meta, sw = oracle.project_pack(W, None, 2, 4, 8)
    D = oracle.unpack(v, meta, out, K, 2, 4, 8)
    sx = np.float32(0.0317)
    acc, Y = oracle.int_linear(X, D, sx, sw, b)
    ref = acc.astype(np.float64) * (np.float64(sx) * sw.astype(np.float64)) + b.astype(np.float64)
    assert np.all(np.abs(Y - ref) <= 1e-6 + 1e-5 * np.abs(ref))
    # exact statement: c rounded once, then one fused multiply-add
    c = (sx * sw).astype(np.float32)
    exact = (acc.astype(np.float64) * c.astype(np.float64) + b.astype(np.float64)).astype(np.float32)
    assert np.array_equal(Y, exact)
    _, Y0 = oracle.int_linear(X, D, sx, sw, None)
    assert np.array_equal(Y0, (acc.astype(np.float64) * c.astype(np.float64)).astype(np.float32))


# ----------------------------------------------------------------------------------------------
# T11: the tie rule (lowest index wins), sign and zero handling
# ----------------------------------------------------------------------------------------------
def test_tie_rule_cases():
    cases = [
        # (row, n, m, expected kept positions per group)
        ([1, 1, 1, 1], 2, 4, [[0, 1]]),
        ([1, -1, 1, -1], 1, 4, [[0]]),
        ([0, 0, 0, 0], 2, 4, [[0, 1]]),
        ([0, -0.0, 0, 5], 2, 4, [[0, 3]]),
        ([1, 2, 2, 1], 2, 4, [[1, 2]]),
        ([1, 2, 1, 2], 1, 4, [[1]]),
        ([2, 1, 1, 2], 2, 4, [[0, 3]]),
        ([1, 2, 1, 1], 2, 4, [[0, 1]]),
        ([3, 3, 3, 3, 3, 3, 3, 3], 4, 8, [[0, 1, 2, 3]]),
        ([1, 3, 1, 3, 1, 3, 1, 3], 2, 8, [[1, 3]]),
        ([1, 3, 1, 3, 1, 3, 1, 3], 1, 8, [[1]]),
        ([0, 0, 0, 0, 0, 0, 0, -1], 2, 8, [[0, 7]]),
        ([5, 0, 0, 0, -5, 0, 0, 5], 2, 8, [[0, 4]]),
    ]
    for row, n, m, expect in cases:
        W = np.array([row], dtype=np.float32)
        v, meta, s = oracle.project_pack(W, None, n, m, 8)
        fb = 2 if m == 4 else 4
        f = _fields(meta[0], len(row) // m * n, fb)
        got = [f[g * n:(g + 1) * n] for g in range(len(row) // m)]
        assert got == expect, (row, n, m, got)


def test_dual_is_added_before_projection():
    # Eq. 3: the projection's argument is W + U, not W.
    W = np.array([[1, 2, 3, 4]], dtype=np.float32)
    U = np.array([[10, 0, 0, -4]], dtype=np.float32)
    v, meta, s = oracle.project_pack(W, U, 2, 4, 8)
    assert _fields(meta[0], 2, 2) == [0, 2]
    assert s[0] == np.float32(11) / np.float32(127)
    assert _codes(v[0], 2, 8) == [127, int(np.rint(np.float32(3) / s[0]))]


def test_round_half_to_even_and_division():
    # scale = 127/127 = 1 -> codes are rne of the values themselves
    W = np.array([[127, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5]], dtype=np.float32)
    v, meta, s = oracle.project_pack(W, None, 4, 4, 8)
    assert s[0] == 1.0
    assert _codes(v[0], 8, 8) == [127, 0, 2, 2, 0, -2, -2, 4]
    # the quotient is a true division: 1/3-type scales
    W = np.array([[3.0, 1.0, 2.0, 0.1]], dtype=np.float32)
    v, meta, s = oracle.project_pack(W, None, 4, 4, 4)
    s_ref = np.float32(3.0) / np.float32(7.0)
    assert s[0] == s_ref
    assert _codes(v[0], 4, 4) == [int(np.rint(x / s_ref)) for x in W[0]]


def test_activation_quantiser():
    Y = wl.normal(np.random.default_rng(95), (7, 33))
    Xq, sx = oracle.quantize_act(Y)
    a = np.abs(Y).max()
    assert sx == a / np.float32(127)
    assert np.array_equal(Xq, np.clip(np.rint(Y / sx), -128, 127).astype(np.int8))
    Xq, sx = oracle.quantize_act(np.zeros((2, 3), np.float32))
    assert sx == 1 and not Xq.any()


def test_nonfinite_flagged():
    W = np.ones((2, 8), np.float32)
    W[1, 3] = np.inf
    with pytest.raises(RuntimeError):
        oracle.project_pack(W, None, 2, 4, 8)


def test_threads_do_not_change_results():
    W = wl.normal(np.random.default_rng(97), (64, 128), 0.02)
    X = wl.random_int8(98, (40, 128))
    oracle.set_threads(1)
    a = oracle.project_pack(W, None, 2, 4, 8)
    D = oracle.unpack(a[0], a[1], 64, 128, 2, 4, 8)
    ya = oracle.int_linear(X, D, 0.01, a[2], None)
    oracle.set_threads(4)
    b = oracle.project_pack(W, None, 2, 4, 8)
    yb = oracle.int_linear(X, D, 0.01, a[2], None)
    oracle.set_threads(1)
    assert all(np.array_equal(p, q) for p, q in zip(a, b))
    assert np.array_equal(ya[0], yb[0]) and np.array_equal(ya[1], yb[1])


# ----------------------------------------------------------------------------------------------
# T-S: storage / FLOP accounting against the numbers printed in Tables 1 and 4
# ----------------------------------------------------------------------------------------------
def _golden():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                rows.append(line)
    return rows


def test_storage_model_matches_paper_tables():
    rows = _golden()
    t1 = {r[1]: float(r[2]) for r in rows if r[0] == "table1_size"}
    # BERT-base encoder linears: 12 x (4 x 768^2 + 2 x 768 x 3072) parameters
    params = 12 * (4 * 768 * 768 + 2 * 768 * 3072)
    mib = lambda bits_per_param: params * bits_per_param / 8 / 2 ** 20
    assert round(mib(32)) == t1["dense_fp32"]
    # fp16 2:4: 16 value bits and 2 index bits per kept value
    assert round(mib(oracle.bits_per_param(2, 4, 16, 2)), 1) == t1["nm24_fp16"]
    assert abs(mib(oracle.bits_per_param(4, 4, 4)) - t1["dense_q4"]) <= 0.5  # 40.5 printed as 41
    # packed sizes the library actually produces agree with the model (2-bit fields at m = 4)
    for n, m, bits in [(2, 4, 8), (2, 4, 4), (1, 4, 8), (1, 4, 4)]:
        vb, mb = oracle.packed_sizes(768, 3072, n, m, bits)
        assert (vb + mb) * 8 == 768 * 3072 * oracle.bits_per_param(n, m, bits, 2)

    cost = {"Q4": oracle.bits_per_param(4, 4, 4), "Q8": oracle.bits_per_param(4, 4, 8),
            "S4": oracle.bits_per_param(2, 4, 4, 2), "S8": oracle.bits_per_param(2, 4, 8, 2)}
    assert cost == {"Q4": 4, "Q8": 8, "S4": 3, "S8": 5}
    units = [1, 1, 1, 1, 4, 4]  # Q, K, V, AttnOut are hidden^2; FFN1, FFN2 are 4 x hidden^2
    for r in rows:
        if r[0] != "table4":
            continue
        cfg, ratio, flop = r[2:8], float(r[8]), r[9]
        bits_total = sum(u * cost[c] for u, c in zip(units, cfg))
        assert round(100 * (1 - bits_total / (12 * 32)), 1) == ratio, r
        if flop != "-":
            sparse_units = sum(u for u, c in zip(units, cfg) if c.startswith("S"))
            assert round(100 * 0.5 * sparse_units / 12, 1) == float(flop), r
    head = {r[1]: float(r[2]) for r in rows if r[0] == "headline"}
    assert 100 * (1 - oracle.bits_per_param(2, 4, 4, 0) / 32) == head["sparse_q4"]
    assert 100 * (1 - oracle.bits_per_param(4, 4, 4) / 32) == head["dense_q4"]


def test_table3_ratios_are_self_consistent():
    rows = _golden()
    fp16, int8, nm = [float(x) for x in next(r for r in rows if r[0] == "table3_b128_s384")[1:]]
    sp = [float(x) for x in next(r for r in rows if r[0] == "table3_speedups")[1:]]
    assert round(fp16 / nm, 1) == sp[0]
    assert round(fp16 / int8, 2) == sp[1]
    assert round(int8 / nm, 2) == sp[2]


# ---- narrow-output forms of the linear layer's result (static-scale int8, bfloat16) -------------------

def test_static_requantiser_closed_forms():
    # exact multiples of a power-of-two scale: the quotient is exact, the code is the clamped multiple
    sy = np.float32(2.0 ** -3)
    k = np.arange(-200, 201, dtype=np.int32)
    q = oracle.requantize_static(k.astype(np.float32) * sy, sy)
    assert np.array_equal(q, np.clip(k, -128, 127).astype(np.int8))
    # exact halves go to the even neighbour (Eq. 5's round read as round-half-to-even)
    halves = (np.arange(-130, 130, dtype=np.float32) + np.float32(0.5)) * sy
    expect = np.array([int(np.clip(2 * round((j + 0.5) / 2), -128, 127)) for j in range(-130, 130)], dtype=np.int8)
    assert np.array_equal(oracle.requantize_static(halves, sy), expect)
    # a scale that is not positive and finite is rejected
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(RuntimeError):
            oracle.requantize_static(np.zeros(4, np.float32), bad)


def test_static_requantiser_properties_and_exact_arithmetic():
    rng = np.random.default_rng(11)
    Y = wl.normal(rng, (4096,), 3.0)
    sy = np.float32(0.0371)
    q = oracle.requantize_static(Y, sy).astype(np.int64)
    inside = np.abs(Y.astype(np.float64)) <= 127.0 * float(sy)
    # within the representable range the reconstruction error is at most half a step (plus the
    # rounding of the fp32 quotient: one part in 2^24 of |y|)
    err = np.abs(Y.astype(np.float64) - float(sy) * q)
    assert np.all(err[inside] <= 0.5 * float(sy) + np.abs(Y[inside]) * 2.0 ** -23)
    assert np.all(q[~inside & (Y > 0)] == 127) and np.all(q[~inside & (Y < 0)] <= -127)
    # monotone in y
    order = np.argsort(Y, kind="stable")
    assert np.all(np.diff(q[order]) >= 0)
    # exact rational arithmetic on the correctly rounded fp32 quotient, element by element
    for y, c in zip(Y[:300], q[:300]):
        quo = Fraction(float(np.float32(y) / sy))        # numpy's IEEE binary32 division
        lo = quo.numerator // quo.denominator
        frac = quo - lo
        r = lo + (1 if (frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1)) else 0)
        assert c == max(-128, min(127, r))
    # with the tensor's own max/127 as the scale it is the dynamic quantiser
    Xq, sx = oracle.quantize_act(Y)
    assert np.array_equal(oracle.requantize_static(Y, sx), Xq)


def test_bf16_rounding_closed_forms_and_library():
    import torch
    one = np.float32(1.0)
    cases = {
        1.0: 0x3F80, -2.75: 0xC030, 0.0: 0x0000,
        float(one + np.float32(2.0 ** -8)): 0x3F80,                          # tie, lower neighbour even
        float(one + np.float32(3 * 2.0 ** -8)): 0x3F82,                      # tie, upper neighbour even
        float(one + np.float32(2.0 ** -8) + np.float32(2.0 ** -20)): 0x3F81,  # just above the tie
        float(one + np.float32(2.0 ** -8) - np.float32(2.0 ** -20)): 0x3F80,  # just below the tie
        float(np.float32(3.3895313892515355e38)): 0x7F7F,                    # largest finite bfloat16 stays
    }
    got = oracle.to_bf16(np.array(list(cases.keys()), dtype=np.float32))
    assert [int(g) for g in got] == list(cases.values())
    # values with at most 8 significant bits are reproduced exactly
    exact = (np.arange(-255, 256, dtype=np.float32) * np.float32(2.0 ** -10))
    back = (oracle.to_bf16(exact).astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(back, exact)
    # half-ulp error bound, monotonicity, agreement with an independent conversion routine
    rng = np.random.default_rng(12)
    Y = np.concatenate([wl.normal(rng, (100000,), 5.0), wl.normal(rng, (1000,), 1e-30), wl.normal(rng, (1000,), 1e30)])
    b = oracle.to_bf16(Y)
    back = (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    normal = np.abs(Y) >= 2.0 ** -126
    assert np.all(np.abs(back - Y)[normal] <= np.abs(Y[normal].astype(np.float64)) * 2.0 ** -8)
    order = np.argsort(Y, kind="stable")
    assert np.all(np.diff(back[order]) >= 0)
    lib = torch.from_numpy(Y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(b, lib)
    with pytest.raises(RuntimeError):
        oracle.to_bf16(np.array([np.inf], np.float32))


# ---- one ADMM projection step with dense outputs (joint projection + dual update) -------------------

@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 4, 8), (2, 8, 4), (4, 8, 8), (4, 4, 8)])
def test_admm_step_is_the_composition_of_the_pinned_pieces(n, m, bits):
    rng = np.random.default_rng(31)
    W, U = wl.normal(rng, (24, 96), 0.02), wl.normal(rng, (24, 96), 0.002)
    Z, Un, s = oracle.admm_step(W, U, n, m, bits)
    V = (W + U).astype(np.float32)
    # scale, sparsity projection and fake-quantiser, each pinned on its own above
    assert np.array_equal(s, oracle.row_scales(V, bits))
    assert np.array_equal(Z, oracle.fake_quant(oracle.project_dense(W, U, n, m), bits, s))
    # the same weights through the packed path: Z = s * unpack(project_pack)
    v, meta, s2 = oracle.project_pack(W, U, n, m, bits)
    D = oracle.unpack(v, meta, 24, 96, n, m, bits)
    assert np.array_equal(s2, s) and np.array_equal(Z, (s[:, None] * D.astype(np.float32)).astype(np.float32))
    # dual update U + W - Z, written here with numpy's own fp32 arithmetic
    assert np.array_equal(Un, (V - Z).astype(np.float32))
    # the constraint holds for Z: at most n nonzeros per group, integer multiples of the row scale within range
    assert ((Z.reshape(24, -1, m) != 0).sum(axis=2) <= n).all()
    codes = Z.astype(np.float64) / s[:, None].astype(np.float64)
    assert np.all(np.abs(codes - np.rint(codes)) < 1e-4) and np.abs(np.rint(codes)).max() <= 2 ** (bits - 1) - 1
    # what is left in the dual: the whole value where pruned, at most half a step (+ rounding) where kept
    kept = Z != 0
    assert np.array_equal(Un[~kept & (np.abs(V) > s[:, None] / 2)], V[~kept & (np.abs(V) > s[:, None] / 2)])
    assert np.all(np.abs(Un[kept]) <= (0.5 * s[:, None] * (1 + 2.0 ** -20) + np.abs(V) * 2.0 ** -23)[kept])


def test_admm_step_fixed_point_and_ste_form():
    rng = np.random.default_rng(32)
    W = wl.normal(rng, (16, 64), 0.02)
    Z, Un, s = oracle.admm_step(W, None, 2, 4, 8)
    # STE forward form: no dual in, none out; same Z
    Z2, none, _ = oracle.admm_step(W, None, 2, 4, 8, want_u=False)
    assert none is None and np.array_equal(Z, Z2)
    # a weight that already meets the constraint stays put: Z(Z) has the same codes and the dual stays ~0
    Zz, Uz, sz = oracle.admm_step(Z, None, 2, 4, 8)
    assert np.array_equal(np.rint(Zz / sz[:, None]), np.rint(Z / s[:, None]))
    assert np.all(np.abs(Uz) <= np.abs(Z) * 2.0 ** -22)
    # W = Z + U_next up to the rounding of the subtraction
    assert np.all(np.abs((Z.astype(np.float64) + Un.astype(np.float64)) - W.astype(np.float64)) <= np.abs(W) * 2.0 ** -23 + 1e-12)
    with pytest.raises(RuntimeError):
        oracle.admm_step(np.array([[np.inf, 0, 0, 0]], np.float32), None, 2, 4, 8)


# ---- group-wise scales (several output channels share one scale) ----------------------------------------

@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 8, 8), (4, 4, 4)])
def test_grouped_scales_reduce_to_the_per_channel_and_whole_matrix_cases(n, m, bits):
    rng = np.random.default_rng(41)
    W, U = wl.normal(rng, (70, 64), 0.02), wl.normal(rng, (70, 64), 0.002)
    V = (W + U).astype(np.float32)
    base = oracle.project_pack(W, U, n, m, bits)
    g1 = oracle.project_pack_grouped(W, U, n, m, bits, 1)
    assert all(np.array_equal(a, b) for a, b in zip(base, g1))          # groups of one channel: the per-channel case
    qmax = np.float32(2 ** (bits - 1) - 1)
    for G in (32, 64, 0, 1000):
        v, meta, s = oracle.project_pack_grouped(W, U, n, m, bits, G)
        rows = 70 if G <= 0 else G
        # one scale per group: the largest row scale of the group (same max, same single division)
        for g0 in range(0, 70, rows):
            grp = slice(g0, min(70, g0 + rows))
            assert np.all(s[grp] == base[2][grp].max())
            assert s[g0] == np.abs(V[grp]).max() / qmax
        # support and metadata do not depend on the scale; the codes are Eq. 5 with the group's scale
        assert np.array_equal(meta, base[1])
        D = oracle.unpack(v, meta, 70, 64, n, m, bits)
        Zs = oracle.project_dense(W, U, n, m)
        assert np.array_equal((s[:, None] * D.astype(np.float32)).astype(np.float32), oracle.fake_quant(Zs, bits, s))
        # the group's largest element still maps to +-qmax, nothing exceeds it
        assert np.abs(D).max() == int(qmax)
    # a row that is small next to its group's maximum loses resolution: fewer distinct codes than with its own scale
    W2 = W.copy(); W2[0] *= 50
    own = oracle.unpack(*oracle.project_pack(W2, None, n, m, bits)[:2], 70, 64, n, m, bits)
    shared = oracle.unpack(*oracle.project_pack_grouped(W2, None, n, m, bits, 32)[:2], 70, 64, n, m, bits)
    assert np.abs(shared[1]).max() < np.abs(own[1]).max()


# ---- ADMM-Dist: the scale that minimises the quantisation distance (Sec. 3.3.1) ---------------------------

def _dist_inputs(kind, seed, out, k):
    rng = np.random.default_rng(seed)
    if kind == "normal":
        return wl.normal(rng, (out, k), 0.02), wl.normal(rng, (out, k), 0.002)
    if kind == "ties":
        return wl.tie_heavy(seed, out, k), None
    return wl.with_outliers(seed, out, k), None


@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 4, 4), (2, 8, 8), (4, 8, 4), (4, 4, 4)])
def test_dist_one_candidate_is_admm_max(n, m, bits):
    W, U = _dist_inputs("normal", 51, 20, 64)
    a, b = oracle.project_pack_dist(W, U, n, m, bits, 1), oracle.project_pack(W, U, n, m, bits)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    E, S, s, c = oracle.dist_search(W, U, n, m, bits, 7)
    assert np.array_equal(S[:, 0], b[2]) and (c < 7).all() and (c >= 0).all()


@pytest.mark.parametrize("kind", ["normal", "ties", "outliers"])
@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 4, 8), (2, 8, 4), (4, 8, 8), (4, 4, 4)])
def test_dist_search_against_exact_rational_arithmetic(kind, n, m, bits):
    """Every candidate's distance recomputed without rounding: numpy's fp32 division and rint give the codes,
    fractions give the sum; the sparsity projection comes from the separately pinned dense routine."""
    out, k, ncand = 6, 32, 32
    W, U = _dist_inputs(kind, 52, out, k)
    E, S, s, c = oracle.dist_search(W, U, n, m, bits, ncand)
    P = oracle.project_dense(W, U, n, m)                     # zero where pruned
    V = W if U is None else (W + U).astype(np.float32)
    qmax = np.float32(2 ** (bits - 1) - 1)
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1) - 1
    for r in range(out):
        a = np.abs(V[r]).max()
        smax = np.float32(1.0) if a == 0 else np.float32(a) / qmax
        exact = []
        for j in range(ncand):
            sj = np.float32(smax * np.float32((64 - j) / 64.0))
            assert S[r, j] == sj
            q = np.clip(np.rint(P[r] / sj), lo, hi).astype(np.int64)     # fp32 quotient, half to even
            e = sum((Fraction(float(x)) - Fraction(float(sj)) * int(qq)) ** 2 for x, qq in zip(P[r], q))
            exact.append(e)
            assert abs(float(e) - E[r, j]) <= 1e-12 * float(e) + 1e-300
        best = min(range(ncand), key=lambda j: (exact[j], j))             # lowest j on equality
        runner = min(exact[j] for j in range(ncand) if j != best)
        if runner == exact[best] or float(runner - exact[best]) > 1e-12 * float(exact[best]):
            assert c[r] == best
        assert exact[c[r]] <= exact[best] * (1 + Fraction(1, 10 ** 12))
        assert s[r] == S[r, c[r]]


@pytest.mark.parametrize("n,m,bits", [(2, 4, 8), (2, 4, 4), (1, 8, 4), (4, 8, 4)])
def test_dist_error_is_the_distance_of_the_packed_output(n, m, bits):
    out, k, ncand = 40, 256, 32
    W, U = _dist_inputs("normal", 53, out, k)
    E, S, s, c = oracle.dist_search(W, U, n, m, bits, ncand)
    P = oracle.project_dense(W, U, n, m).astype(np.float64)
    for packed, col in ((oracle.project_pack_dist(W, U, n, m, bits, ncand), c),
                        (oracle.project_pack(W, U, n, m, bits), np.zeros(out, np.int64))):
        v, meta, sc = packed
        D = oracle.unpack(v, meta, out, k, n, m, bits).astype(np.float64)
        dist = ((sc.astype(np.float64)[:, None] * D - P) ** 2).sum(axis=1)
        assert np.allclose(dist, E[np.arange(out), col], rtol=1e-11, atol=0)
    # never worse than ADMM-Max, and the minimum over the sweep
    assert (E[np.arange(out), c] <= E[:, 0]).all() and np.array_equal(E[np.arange(out), c], E.min(axis=1))
    assert np.array_equal(c, E.argmin(axis=1))                # numpy's argmin: first minimum
    # the metadata (support) does not depend on the scale
    assert np.array_equal(oracle.project_pack_dist(W, U, n, m, bits, ncand)[1], oracle.project_pack(W, U, n, m, bits)[1])
    # handing the chosen scales in gives the same bytes
    a, b = oracle.project_pack_dist(W, U, n, m, bits, ncand), oracle.project_pack_scaled(W, U, n, m, bits, s)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_dist_pays_at_four_bits_and_not_at_eight():
    """Gaussian rows of 1024: with 7 levels a side the best scale clips the tail (c well below 1); with 127 the
    row maximum (about 3.2 sigma) is already near the best range."""
    W, _ = _dist_inputs("normal", 54, 48, 1024)
    E4, _, _, c4 = oracle.dist_search(W, None, 2, 4, 4, 32)
    E8, _, _, c8 = oracle.dist_search(W, None, 2, 4, 8, 32)
    assert (c4 >= 4).mean() > 0.9 and (E4[np.arange(48), c4] < 0.9 * E4[:, 0]).mean() > 0.9
    assert (c8 <= 3).all() and (E8[np.arange(48), c8] > 0.75 * E8[:, 0]).all()
    assert c4.max() < 31                                        # the sweep's range contains the minimum


def test_dist_power_of_two_invariance_zero_rows_and_arguments():
    W, U = _dist_inputs("outliers", 55, 12, 64)                 # has an all-zero row and zero groups
    base = oracle.project_pack_dist(W, None, 2, 4, 4, 32)
    E, S, s, c = oracle.dist_search(W, None, 2, 4, 4, 32)
    z = 12 // 2
    assert c[z] == 0 and s[z] == 1.0 and (E[z] == 0).all() and not base[0][z].any()
    for p in (-20, 7):
        f = np.float32(2.0 ** p)
        v, meta, sc = oracle.project_pack_dist(W * f, None, 2, 4, 4, 32)
        nz = np.arange(12) != z
        assert np.array_equal(v, base[0]) and np.array_equal(meta, base[1]) and np.array_equal(sc[nz], base[2][nz] * f)
    for bad in (0, 33):
        with pytest.raises(RuntimeError):
            oracle.dist_search(W, None, 2, 4, 4, bad)
    # clipping reaches the most negative code, which ADMM-Max never produces
    Wn = np.zeros((1, 64), np.float32); Wn[0, ::2] = 0.01; Wn[0, 0] = -0.05; Wn[0, 2] = 0.05
    v, meta, sc = oracle.project_pack_dist(Wn, None, 2, 4, 4, 32)
    D = oracle.unpack(v, meta, 1, 64, 2, 4, 4)
    assert sc[0] < np.float32(0.05) / 7 and D.min() == -8 and D.max() == 7


@pytest.mark.parametrize("n,m,bits", [(2, 4, 4), (1, 4, 8), (4, 4, 4)])
def test_admm_step_dist_is_the_composition(n, m, bits):
    W, U = _dist_inputs("normal", 56, 16, 128)
    Z, Un, s = oracle.admm_step_dist(W, U, n, m, bits, 32)
    v, meta, s2 = oracle.project_pack_dist(W, U, n, m, bits, 32)
    D = oracle.unpack(v, meta, 16, 128, n, m, bits)
    V = (W + U).astype(np.float32)
    assert np.array_equal(s, s2) and np.array_equal(Z, (s[:, None] * D.astype(np.float32)).astype(np.float32))
    assert np.array_equal(Un, (V - Z).astype(np.float32))
    assert np.array_equal(Z, oracle.fake_quant(oracle.project_dense(W, U, n, m), bits, s))
