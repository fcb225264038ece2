"""GPU parity on the heterogeneous encoder GEMM chain and on full-size shapes.

Chain wiring (one encoder layer): h -> QKV -> take the V slice as stand-in for the attention
context -> output projection -> FFN1 -> FFN2 -> next layer; between GEMMs the fp32 result is
re-quantised per tensor to int8.  Every GEMM draws its weight format from
{dense int8, 2:4 int8, 2:4 int4, 1:4 int8, 4:8 int8}.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


def _oracle_chain(modes, h0, weights, hidden):
    """-> list of (Xq_in, sx_in, Y) per GEMM, free running."""
    trace = []
    Xq, sx = oracle.quantize_act(h0)
    for layer, wrow in zip(modes, weights):
        for g, (mode, (W, b)) in enumerate(zip(layer, wrow)):
            n, m, bits = wl.CHAIN_MODES[mode]
            v, meta, s = oracle.project_pack(W, None, n, m, bits)
            D = oracle.unpack(v, meta, W.shape[0], W.shape[1], n, m, bits)
            _, Y = oracle.int_linear(Xq, D, sx, s, b, want_acc=False)
            trace.append((Xq, sx, Y))
            nxt = Y[:, 2 * hidden:] if g == 0 else Y  # QKV: only the V slice feeds the next GEMM
            Xq, sx = oracle.quantize_act(np.ascontiguousarray(nxt))
    return trace


def _gpu_chain(modes, h0, weights, hidden, teacher=None):
    """Runs the chain through the C ABI.  teacher: oracle trace whose int8 inputs are fed to every
    GEMM instead of the GPU's own (teacher forcing).  -> list of (Xq_in, sx_in, Y) as numpy."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    T = h0.shape[0]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def requant(Yd):
        amax = torch.zeros(1, dtype=torch.float32, device=DEV)
        sx = torch.empty(1, dtype=torch.float32, device=DEV)
        Xq = torch.empty(Yd.shape, dtype=torch.int8, device=DEV)
        nm.nm_absmax(Yd, Yd.numel(), amax)
        nm.nm_quantize_act(Yd, Yd.numel(), amax, Xq, sx)
        return Xq, sx

    Xq, sx = requant(to_dev(h0))
    trace, step = [], 0
    for layer, wrow in zip(modes, weights):
        for g, (mode, (W, b)) in enumerate(zip(layer, wrow)):
            n, m, bits = wl.CHAIN_MODES[mode]
            out, k = W.shape
            vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
            values = torch.empty(vb, dtype=torch.uint8, device=DEV)
            meta = torch.empty(max(mb // 4, 1), dtype=torch.int32, device=DEV)
            scales = torch.empty(out, dtype=torch.float32, device=DEV)
            nm.nm_project_pack(to_dev(W), None, out, k, n, m, bits, values, meta if mb else None, scales, status)
            if teacher is not None:
                Xq, sx = to_dev(teacher[step][0]), to_dev(np.array([teacher[step][1]], np.float32))
            Y = torch.empty((T, out), dtype=torch.float32, device=DEV)
            amax = torch.zeros(1, dtype=torch.float32, device=DEV)
            nm.nm_int_linear_dsx(Xq, T, nm.make_packed(out, k, n, m, bits, values, meta if mb else None), sx, scales,
                                 to_dev(b), Y, amax, status=status)
            trace.append((Xq.cpu().numpy(), float(sx.item()), Y.cpu().numpy()))
            if g == 0:
                Xq, sx = requant(Y[:, 2 * hidden:].contiguous())  # a copy of the V slice, no arithmetic
            else:  # the GEMM's own running max|Y| feeds the quantiser
                sx = torch.empty(1, dtype=torch.float32, device=DEV)
                Xq = torch.empty(Y.shape, dtype=torch.int8, device=DEV)
                nm.nm_quantize_act(Y, Y.numel(), amax, Xq, sx)
            step += 1
    assert nm.nm_poll_status(status) == nm.NM_OK
    return trace


def test_heterogeneous_chain_matches_oracle():
    from gpu_util import assert_close
    oracle.set_threads(oracle.max_threads())
    hidden, T, layers = 768, 768, 12          # 2 sequences of 384 tokens; all 12 layers, 48 GEMMs
    modes, h0, weights = wl.chain_case(4, layers=layers, tokens=T)
    assert set(np.unique(modes)) == set(range(len(wl.CHAIN_MODES)))  # every format is drawn
    ref = _oracle_chain(modes, h0, weights, hidden)
    forced = _gpu_chain(modes, h0, weights, hidden, teacher=ref)
    for i, ((xr, sr, yr), (xg, sg, yg)) in enumerate(zip(ref, forced)):
        assert_close(yg, yr)
        assert np.array_equal(yg, yr), f"GEMM {i}: fp32 outputs not identical under teacher forcing"
    free = _gpu_chain(modes, h0, weights, hidden)
    for i, ((xr, sr, yr), (xg, sg, yg)) in enumerate(zip(ref, free)):
        assert np.array_equal(xg, xr), f"GEMM {i}: int8 input differs in {(xg != xr).sum()} places"
        assert sg == sr, f"GEMM {i}: activation scale differs"
        assert_close(yg, yr)


def test_chain_full_size_matches_oracle():
    """Two encoder layers (8 GEMMs, every weight format of the seed's draw) at the benchmark's 6144 tokens, free
    running: every int8 input, every activation scale and every fp32 output of every GEMM against the oracle, and the
    run repeated bit for bit."""
    from gpu_util import assert_close
    oracle.set_threads(oracle.max_threads())
    hidden, T = 768, 6144                    # batch 16 x sequence 384
    modes, h0, weights = wl.chain_case(4, layers=2, tokens=T)
    ref = _oracle_chain(modes, h0, weights, hidden)
    a = _gpu_chain(modes, h0, weights, hidden)
    b = _gpu_chain(modes, h0, weights, hidden)
    for i, ((xr, sr, yr), (xa, sa, ya), (xb, sb, yb)) in enumerate(zip(ref, a, b)):
        assert np.array_equal(xa, xb) and sa == sb and np.array_equal(ya, yb), f"GEMM {i}: two runs differ"
        assert np.array_equal(xa, xr), f"GEMM {i}: int8 input differs in {(xa != xr).sum()} places"
        assert sa == sr, f"GEMM {i}: activation scale differs"
        assert_close(ya, yr)
        assert np.array_equal(ya, yr), f"GEMM {i}: fp32 outputs not identical"


@pytest.mark.parametrize("name,k,out", wl.BERT_LARGE_GEMMS)
@pytest.mark.parametrize("bits", [8, 4])
def test_bert_large_full_size(name, k, out, bits):
    """16384 tokens, 2:4 weights, the launch configuration the benchmark times: every output of the launch
    against the oracle (a guard row past the last token stays untouched)."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    oracle.set_threads(oracle.max_threads())
    T = 16384
    rng = np.random.default_rng([2, k, out, bits])
    W = wl.normal(rng, (out, k), wl.W_STD)
    b = wl.normal(rng, (out,), wl.W_STD)
    Xq = wl.random_int8([5, k, out], (T, k))
    v, meta, s = oracle.project_pack(W, None, 2, 4, bits)
    D = oracle.unpack(v, meta, out, k, 2, 4, bits)
    Y = torch.full((T + 1, out), float("nan"), dtype=torch.float32, device=DEV)
    vd, md, sd = to_dev(v.reshape(-1)), to_dev(meta.reshape(-1).view(np.int32)), to_dev(s)
    nm.nm_int_linear(to_dev(Xq), T, nm.make_packed(out, k, 2, 4, bits, vd, md), 0.03, sd, to_dev(b), Y)
    assert nm.nm_poll_status() == nm.NM_OK
    Yh = Y.cpu().numpy()
    assert np.isnan(Yh[T]).all(), "Y written past the last token"
    _, Yr = oracle.int_linear(Xq, D, 0.03, s, b, want_acc=False)
    assert np.array_equal(Yh[:T], Yr), f"{(Yh[:T] != Yr).sum()} of {Yr.size} outputs differ"


@pytest.mark.parametrize("name,k,out", wl.BERT_LARGE_GEMMS)
def test_bert_large_full_size_narrow_outputs(name, k, out):
    """16384 tokens, 2:4 int8 weights, the launch configurations `bench.py --out int8 | bf16` times (sixteen epilogue warps
    on the resident-weight kernel, shared staging tiles on the 512-channel kernel): every int8 code and every bfloat16
    pattern of the launch against the oracle."""
    from gpu_util import PackedOnDevice, gpu_int_linear_q8, gpu_int_linear_bf16
    oracle.set_threads(oracle.max_threads())
    T = 16384
    rng = np.random.default_rng([6, k, out])
    W = wl.normal(rng, (out, k), wl.W_STD)
    b = wl.normal(rng, (out,), wl.W_STD)
    Xq = wl.random_int8([7, k, out], (T, k))
    v, meta, s = oracle.project_pack(W, None, 2, 4, 8)
    D = oracle.unpack(v, meta, out, k, 2, 4, 8)
    _, Yr = oracle.int_linear(Xq, D, 0.03, s, b, want_acc=False)
    packed = PackedOnDevice(v, meta, s, out, k, 2, 4, 8)
    sy = np.float32(np.abs(Yr).max()) / np.float32(100.0)       # a few outputs clamp
    got = gpu_int_linear_q8(Xq, packed, 0.03, b, sy)
    ref = oracle.requantize_static(Yr, sy)
    assert np.array_equal(got, ref), f"{(got != ref).sum()} of {ref.size} int8 codes differ"
    got = gpu_int_linear_bf16(Xq, packed, 0.03, b)
    ref = oracle.to_bf16(Yr)
    assert np.array_equal(got, ref), f"{(got != ref).sum()} of {ref.size} bfloat16 patterns differ"


def test_pack_sweep_full_size_batched():
    """One batched launch over a full BERT-large layer (2:4, 8 bit) against the oracle, bit for bit."""
    import paper_2206_15014_b200 as nm
    from gpu_util import DEV, to_dev
    oracle.set_threads(oracle.max_threads())
    jobs, refs = [], []
    for i, (name, k, out) in enumerate(wl.BERT_LARGE_GEMMS):
        W, U = wl.pack_sweep_matrix(3, i, out, k)
        vb, mb = nm.nm_packed_sizes(out, k, 2, 4, 8)
        jobs.append((to_dev(W), to_dev(U), 2, 4, 8, torch.zeros(vb, dtype=torch.uint8, device=DEV),
                     torch.zeros(mb // 4, dtype=torch.int32, device=DEV), torch.zeros(out, dtype=torch.float32, device=DEV)))
        refs.append(oracle.project_pack(W, U, 2, 4, 8))
    ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    nm.nm_project_pack_batched(nm.make_pack_jobs(jobs), len(jobs), ws, ws_bytes, status)
    assert nm.nm_poll_status(status) == nm.NM_OK
    for job, (v, meta, s) in zip(jobs, refs):
        assert np.array_equal(job[5].cpu().numpy().reshape(v.shape), v)
        assert np.array_equal(job[6].cpu().numpy().view(np.uint32).reshape(meta.shape), meta)
        assert np.array_equal(job[7].cpu().numpy(), s)
