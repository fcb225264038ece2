"""GPU parity of kernels that consume each other's results back to back in one stream.

The CTA-pair GEMM is launched as a programmatic dependent of the kernel in front of it, so its set-up runs
while that kernel drains; it must still see everything that kernel wrote.  Here the projection kernel's
packed weights feed a GEMM whose int8 result feeds the next GEMM, with no host synchronisation in between,
several times over poisoned buffers, and the end result is compared with the oracle's.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


def test_pack_then_two_dependent_gemms_without_host_syncs():
    import paper_2206_15014_b200 as nm
    from gpu_util import to_dev, DEV, assert_close
    T, K, H, out = 4096, 1024, 1024, 1024   # 88 pair tiles per GEMM: the CTA-pair kernel
    rng = np.random.default_rng(61)
    W1, b1 = wl.normal(rng, (H, K), 0.02), wl.normal(rng, (H,), 0.02)
    W2, b2 = wl.normal(rng, (out, H), 0.02), wl.normal(rng, (out,), 0.02)
    Xq, sx = oracle.quantize_act(wl.normal(rng, (T, K)))
    oracle.set_threads(oracle.max_threads())
    v1, m1, s1 = oracle.project_pack(W1, None, 2, 4, 8)
    v2, m2, s2 = oracle.project_pack(W2, None, 2, 4, 8)
    _, Y1 = oracle.int_linear(Xq, oracle.unpack(v1, m1, H, K, 2, 4, 8), sx, s1, b1, want_acc=False)
    sy = np.float32(np.abs(Y1).max()) / np.float32(127.0)
    H1 = oracle.requantize_static(Y1, sy)
    _, Y2 = oracle.int_linear(H1, oracle.unpack(v2, m2, out, H, 2, 4, 8), sy, s2, b2, want_acc=False)

    Xd, W1d, W2d, b1d, b2d = to_dev(Xq), to_dev(W1), to_dev(W2), to_dev(b1), to_dev(b2)
    def packed_bufs(o, k):
        vb, mb = nm.nm_packed_sizes(o, k, 2, 4, 8)
        return (torch.empty(vb, dtype=torch.uint8, device=DEV), torch.empty(mb // 4, dtype=torch.int32, device=DEV),
                torch.empty(o, dtype=torch.float32, device=DEV))
    p1, p2 = packed_bufs(H, K), packed_bufs(out, H)
    Yq1 = torch.empty((T, H), dtype=torch.int8, device=DEV)
    Y = torch.empty((T, out), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    d1 = nm.make_packed(H, K, 2, 4, 8, p1[0], p1[1])
    d2 = nm.make_packed(out, H, 2, 4, 8, p2[0], p2[1])
    for rep in range(4):
        for t in (*p1, *p2, Yq1, Y):                      # stale results must not survive
            t.fill_(1 if t.dtype != torch.float32 else float("nan"))
        nm.nm_project_pack(W2d, None, out, H, 2, 4, 8, *p2, status)
        nm.nm_project_pack(W1d, None, H, K, 2, 4, 8, *p1, status)                     # kernel in front of GEMM 1
        nm.nm_int_linear_q8(Xd, T, d1, float(sx), p1[2], b1d, float(sy), Yq1, status=status)   # reads what it wrote
        nm.nm_int_linear(Yq1, T, d2, float(sy), p2[2], b2d, Y, status=status)          # reads GEMM 1's result
        assert nm.nm_poll_status(status) == nm.NM_OK
        assert np.array_equal(p1[0].cpu().numpy().reshape(v1.shape), v1), f"round {rep}: packed weights"
        assert np.array_equal(Yq1.cpu().numpy(), H1), f"round {rep}: first layer"
        assert_close(Y.cpu().numpy(), Y2)
        assert np.array_equal(Y.cpu().numpy(), Y2), f"round {rep}: second layer"
