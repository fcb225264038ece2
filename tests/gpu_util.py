"""Helpers for the GPU parity tests: marshal numpy inputs to the C-ABI calls and back."""
import numpy as np
import torch

import paper_2206_15014_b200 as nm

DEV = torch.device("cuda:0")


def to_dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def gpu_project_pack(W, U, n, m, bits):
    """-> (values u8 [out,row_bytes], meta u32 [out,row_words], scales f32, status code)."""
    out, k = W.shape
    vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
    Wd, Ud = to_dev(W), to_dev(U)
    values = torch.full((max(vb, 1) + 64,), 0xAB, dtype=torch.uint8, device=DEV)  # canary tail
    meta = torch.full((max(mb // 4, 1) + 16,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
    scales = torch.empty(max(out, 1), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_project_pack(Wd, Ud, out, k, n, m, bits, values, meta if mb else None, scales, status)
    rc = nm.nm_poll_status(status)
    v = values.cpu().numpy()
    mt = meta.cpu().numpy().view(np.uint32)
    assert (v[vb:] == 0xAB).all(), "values written past the end"
    assert (mt[mb // 4:] == 0x5A5A5A5A).all(), "metadata written past the end"
    return (v[:vb].reshape(out, -1) if out else v[:0].reshape(0, 0),
            mt[:mb // 4].reshape(out, -1) if out and mb else mt[:0].reshape(out, 0),
            scales.cpu().numpy()[:out], rc)


class PackedOnDevice:
    """Packed weights uploaded from oracle arrays (teacher-forced inputs for the GEMM tests)."""

    def __init__(self, values, meta, scales, out, k, n, m, bits):
        self.values = to_dev(values.reshape(-1))
        self.meta = to_dev(meta.reshape(-1).view(np.int32)) if n != m else None
        self.scales = to_dev(scales)
        self.out, self.k, self.n, self.m, self.bits = out, k, n, m, bits
        self.desc = nm.make_packed(out, k, n, m, bits, self.values, self.meta)


def gpu_int_linear(Xq, packed, sx, bias, want_acc=True):
    T = Xq.shape[0]
    Xd = to_dev(Xq)
    bd = to_dev(bias)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    Y = torch.full((T + 1, packed.out), float("nan"), dtype=torch.float32, device=DEV)
    nm.nm_int_linear(Xd, T, packed.desc, float(sx), packed.scales, bd, Y, status=status)
    acc = None
    if want_acc:
        acc = torch.full((T + 1, packed.out), -7, dtype=torch.int32, device=DEV)
        nm.nm_int_linear_acc(Xd, T, packed.desc, acc, status=status)
    rc = nm.nm_poll_status(status)
    assert rc == nm.NM_OK, nm.nm_strerror(rc)
    Yh = Y.cpu().numpy()
    assert np.isnan(Yh[T]).all(), "Y written past the last token"
    if want_acc:
        acch = acc.cpu().numpy()
        assert (acch[T] == -7).all()
        acc = acch[:T]
    return acc, Yh[:T]


def assert_close(Y, Y_ref):
    err = np.abs(Y.astype(np.float64) - Y_ref.astype(np.float64))
    tol = 1e-6 + 1e-5 * np.abs(Y_ref.astype(np.float64))
    bad = err > tol
    assert not bad.any(), f"{bad.sum()} of {bad.size} outside 1e-5 rel / 1e-6 abs; max err {err.max()}"


def gpu_int_linear_q8(Xq, packed, sx, bias, sy):
    """Static-scale int8 output of the layer; one guard row past the last token must stay untouched."""
    T = Xq.shape[0]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    Yq = torch.full((T + 1, packed.out), 99, dtype=torch.int8, device=DEV)
    nm.nm_int_linear_q8(to_dev(Xq), T, packed.desc, float(sx), packed.scales, to_dev(bias), float(sy), Yq, status=status)
    rc = nm.nm_poll_status(status)
    assert rc == nm.NM_OK, nm.nm_strerror(rc)
    h = Yq.cpu().numpy()
    assert (h[T] == 99).all(), "Yq written past the last token"
    return h[:T]


def gpu_int_linear_bf16(Xq, packed, sx, bias):
    """bfloat16 output of the layer as uint16 bit patterns."""
    T = Xq.shape[0]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    Yb = torch.full((T + 1, packed.out), 0x7FC1, dtype=torch.int16, device=DEV)
    nm.nm_int_linear_bf16(to_dev(Xq), T, packed.desc, float(sx), packed.scales, to_dev(bias), Yb, status=status)
    rc = nm.nm_poll_status(status)
    assert rc == nm.NM_OK, nm.nm_strerror(rc)
    h = Yb.cpu().numpy().view(np.uint16)
    assert (h[T] == 0x7FC1).all(), "Y written past the last token"
    return h[:T]
