"""CPU oracle for the N:M low-bit path -- TEST INFRASTRUCTURE, not product code.

Thin ctypes access to ``nm_oracle.c`` (plain scalar C written from the paper).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and this package imports nothing of
the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nm_oracle.c")
_LIB = os.path.join(_HERE, "libnm_oracle.so")


def build(force: bool = False) -> str:
    """Compile nm_oracle.c with gcc (no fast-math, no contraction). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
             "-fno-fast-math", "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_bits_per_param.restype = ctypes.c_double
        _lib.oracle_bits_per_param.argtypes = [ctypes.c_int] * 4
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with oracle status {rc}")


def set_threads(t: int) -> None:
    lib().oracle_set_threads(int(t))


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def packed_sizes(out, inn, n, m, bits):
    vb, mb = ctypes.c_size_t(), ctypes.c_size_t()
    _chk(lib().oracle_packed_sizes(out, inn, n, m, bits, ctypes.byref(vb), ctypes.byref(mb)),
         "oracle_packed_sizes")
    return vb.value, mb.value


def project_pack(W, U, n, m, bits):
    """-> (values u8 [out, row_bytes], meta u32 [out, row_words], scales f32 [out])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    out, inn = W.shape
    vb, mb = packed_sizes(out, inn, n, m, bits)
    values = np.zeros((out, vb // max(out, 1)), dtype=np.uint8)
    meta = np.zeros((out, mb // 4 // max(out, 1)), dtype=np.uint32)
    scales = np.zeros(out, dtype=np.float32)
    _chk(lib().oracle_project_pack(_p(W), _p(U), out, inn, n, m, bits, _p(values),
                                   _p(meta) if mb else None, _p(scales)), "oracle_project_pack")
    return values, meta, scales


def unpack(values, meta, out, inn, n, m, bits):
    """-> dense int8 codes [out, in], zero where pruned."""
    values = np.ascontiguousarray(values, dtype=np.uint8)
    meta = None if (meta is None or n == m) else np.ascontiguousarray(meta, dtype=np.uint32)
    Wq = np.zeros((out, inn), dtype=np.int8)
    _chk(lib().oracle_unpack(_p(values), _p(meta), out, inn, n, m, bits, _p(Wq)), "oracle_unpack")
    return Wq


def project_pack_grouped(W, U, n, m, bits, group_rows):
    """As project_pack with one scale per group of `group_rows` output channels (<= 0: whole matrix)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    out, inn = W.shape
    vb, mb = packed_sizes(out, inn, n, m, bits)
    values = np.zeros((out, vb // max(out, 1)), dtype=np.uint8)
    meta = np.zeros((out, mb // 4 // max(out, 1)), dtype=np.uint32)
    scales = np.zeros(out, dtype=np.float32)
    _chk(lib().oracle_project_pack_grouped(_p(W), _p(U), out, inn, n, m, bits, int(group_rows), _p(values),
                                           _p(meta) if mb else None, _p(scales)), "oracle_project_pack_grouped")
    return values, meta, scales


def dist_search(W, U, n, m, bits, ncand):
    """ADMM-Dist candidate sweep -> (E f64 [out, ncand], S f32 [out, ncand], scales f32 [out], cand i32 [out])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    out, inn = W.shape
    E = np.zeros((out, ncand), dtype=np.float64)
    S = np.zeros((out, ncand), dtype=np.float32)
    scales = np.zeros(out, dtype=np.float32)
    cand = np.zeros(out, dtype=np.int32)
    _chk(lib().oracle_dist_search(_p(W), _p(U), out, inn, n, m, bits, int(ncand), _p(E), _p(S), _p(scales),
                                  _p(cand)), "oracle_dist_search")
    return E, S, scales, cand


def _packed_out(out, inn, n, m, bits):
    vb, mb = packed_sizes(out, inn, n, m, bits)
    return (np.zeros((out, vb // max(out, 1)), dtype=np.uint8),
            np.zeros((out, mb // 4 // max(out, 1)), dtype=np.uint32), np.zeros(out, dtype=np.float32), mb)


def project_pack_scaled(W, U, n, m, bits, given_scales):
    """As project_pack with the per-channel scales handed in."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    given = np.ascontiguousarray(given_scales, dtype=np.float32)
    out, inn = W.shape
    assert given.shape == (out,)
    values, meta, scales, mb = _packed_out(out, inn, n, m, bits)
    _chk(lib().oracle_project_pack_scaled(_p(W), _p(U), out, inn, n, m, bits, _p(given), _p(values),
                                          _p(meta) if mb else None, _p(scales)), "oracle_project_pack_scaled")
    return values, meta, scales


def project_pack_dist(W, U, n, m, bits, ncand):
    """As project_pack with the ADMM-Dist scale (candidate sweep of dist_search)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    out, inn = W.shape
    values, meta, scales, mb = _packed_out(out, inn, n, m, bits)
    _chk(lib().oracle_project_pack_dist(_p(W), _p(U), out, inn, n, m, bits, int(ncand), _p(values),
                                        _p(meta) if mb else None, _p(scales)), "oracle_project_pack_dist")
    return values, meta, scales


def admm_step_dist(W, U, n, m, bits, ncand, want_u=True):
    """admm_step with the ADMM-Dist scale."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    Z = np.zeros_like(W)
    Un = np.zeros_like(W) if want_u else None
    s = np.zeros(W.shape[0], dtype=np.float32)
    _chk(lib().oracle_admm_step_dist(_p(W), _p(U), W.shape[0], W.shape[1], n, m, bits, int(ncand), _p(Z),
                                     _p(Un), _p(s)), "oracle_admm_step_dist")
    return Z, Un, s


def project_dense(W, U, n, m):
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    Z = np.zeros_like(W)
    _chk(lib().oracle_project_dense(_p(W), _p(U), W.shape[0], W.shape[1], n, m, _p(Z)),
         "oracle_project_dense")
    return Z


def row_scales(V, bits):
    V = np.ascontiguousarray(V, dtype=np.float32)
    s = np.zeros(V.shape[0], dtype=np.float32)
    _chk(lib().oracle_row_scales(_p(V), V.shape[0], V.shape[1], bits, _p(s)), "oracle_row_scales")
    return s


def fake_quant(Z, bits, scales):
    Z = np.ascontiguousarray(Z, dtype=np.float32)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    Zq = np.zeros_like(Z)
    _chk(lib().oracle_fake_quant(_p(Z), Z.shape[0], Z.shape[1], bits, _p(scales), _p(Zq)),
         "oracle_fake_quant")
    return Zq


def admm_step(W, U, n, m, bits, want_u=True):
    """-> (Z f32 like W, U_next f32 | None, scales f32 [out]): joint projection as dense fp32 + dual update."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    U = None if U is None else np.ascontiguousarray(U, dtype=np.float32)
    Z = np.zeros_like(W)
    Un = np.zeros_like(W) if want_u else None
    s = np.zeros(W.shape[0], dtype=np.float32)
    _chk(lib().oracle_admm_step(_p(W), _p(U), W.shape[0], W.shape[1], n, m, bits, _p(Z), _p(Un), _p(s)),
         "oracle_admm_step")
    return Z, Un, s


def int_linear(X, Wq, sx, sw, bias, want_acc=True, want_y=True):
    """X int8 [T, in], Wq int8 dense [out, in] -> (acc int32 [T, out] | None, Y f32 [T, out] | None)."""
    X = np.ascontiguousarray(X, dtype=np.int8)
    Wq = np.ascontiguousarray(Wq, dtype=np.int8)
    T, inn = X.shape
    out = Wq.shape[0]
    assert Wq.shape[1] == inn
    sw = np.ascontiguousarray(sw, dtype=np.float32)
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    acc = np.zeros((T, out), dtype=np.int32) if want_acc else None
    Y = np.zeros((T, out), dtype=np.float32) if want_y else None
    _chk(lib().oracle_int_linear(_p(X), T, _p(Wq), out, inn, ctypes.c_float(float(sx)), _p(sw),
                                 _p(bias), _p(acc), _p(Y)), "oracle_int_linear")
    return acc, Y


def int_linear_kept(X, values, meta, out, inn, n, m, bits):
    X = np.ascontiguousarray(X, dtype=np.int8)
    values = np.ascontiguousarray(values, dtype=np.uint8)
    meta = None if (meta is None or n == m) else np.ascontiguousarray(meta, dtype=np.uint32)
    acc = np.zeros((X.shape[0], out), dtype=np.int32)
    _chk(lib().oracle_int_linear_kept(_p(X), X.shape[0], _p(values), _p(meta), out, inn, n, m,
                                      bits, _p(acc)), "oracle_int_linear_kept")
    return acc


def quantize_act(Y):
    """-> (Xq int8 like Y, sx float32 scalar)."""
    Y = np.ascontiguousarray(Y, dtype=np.float32)
    Xq = np.zeros(Y.shape, dtype=np.int8)
    sx = ctypes.c_float()
    _chk(lib().oracle_quantize_act(_p(Y), ctypes.c_size_t(Y.size), _p(Xq), ctypes.byref(sx)),
         "oracle_quantize_act")
    return Xq, np.float32(sx.value)


def requantize_static(Y, sy):
    """Eq. 5 with b = 8 and a given scale: -> int8 like Y."""
    Y = np.ascontiguousarray(Y, dtype=np.float32)
    Yq = np.zeros(Y.shape, dtype=np.int8)
    _chk(lib().oracle_requantize_static(_p(Y), ctypes.c_size_t(Y.size), ctypes.c_float(float(sy)), _p(Yq)),
         "oracle_requantize_static")
    return Yq


def to_bf16(Y):
    """fp32 -> bfloat16 bit patterns (uint16 like Y), round to nearest even."""
    Y = np.ascontiguousarray(Y, dtype=np.float32)
    out = np.zeros(Y.shape, dtype=np.uint16)
    _chk(lib().oracle_to_bf16(_p(Y), ctypes.c_size_t(Y.size), _p(out)), "oracle_to_bf16")
    return out


def bits_per_param(n, m, bits, index_bits=-1):
    return float(lib().oracle_bits_per_param(n, m, bits, index_bits))
