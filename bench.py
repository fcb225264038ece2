#!/usr/bin/env python
"""Benchmark of the N:M low-bit hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
  (1) projection + quantise + pack (2:4, 8 bit) of the four linear weights of one BERT-large
      encoder layer (W ~ N(0,0.02) plus ADMM dual U ~ N(0,0.002)), one batched launch;
  (2) the four integer 2:4 GEMMs of that layer (QKV 1024->3072, out 1024->1024, FFN1 1024->4096,
      FFN2 4096->1024) at 16384 tokens, int8 activations, fp32 bias + dequantisation epilogue.
`value` is the dense-equivalent integer throughput of the step's GEMMs (2 * T * K * out summed over
the four shapes) divided by the whole step time, in TOPS.  Per-kernel figures (GEMM TOPS per shape,
projection/pack GB/s on the full 24-layer sweep) ride along in `kernels`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 (launched under torchrun): every rank runs the same per-GPU workload on its own data, no
data-path collective (weak scaling); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

TOKENS = 16384
PATTERN = (2, 4, 8)
NOMINAL_SPARSE_INT8_TOPS = 9000.0   # vendor figure for 2:4 INT8 on one B200 (dense 4500)
NOMINAL_HBM_GBS = 8000.0
METRIC = "2:4-sparse INT8 GEMM dense-equivalent TOPS over one hot-path step (pack + 4 GEMMs)"
WORKLOAD = "BERT-large encoder-layer GEMMs (QKV/out/FFN1/FFN2, hidden 1024) at 16384 tokens, 2:4 int8 weights"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def gemm_ops(tokens, k, out):
    return 2.0 * tokens * k * out


def gemm_bytes(tokens, k, out, n=2, m=4, bits=8, ybytes=4):
    """Algorithmic HBM bytes of one GEMM launch: X + packed values + metadata + scales/bias + Y."""
    fb = 2 if m == 4 else 4
    vals = out * (k // m) * n * bits / 8
    meta = 0 if n == m else out * (k // m) * n * fb / 8
    return tokens * k + vals + meta + 8 * out + float(ybytes) * tokens * out


def pack_bytes(out, k, n, m, bits, with_u=True):
    """Algorithmic HBM bytes of packing one matrix: W (+U) read, values + metadata + scales written."""
    fb = 2 if m == 4 else 4
    vals = out * (k // m) * n * bits / 8
    meta = 0 if n == m else out * (k // m) * n * fb / 8
    return out * k * 4.0 * (2 if with_u else 1) + vals + meta + 4 * out


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        fd, self.path = tempfile.mkstemp(suffix=".csv")
        os.close(fd)
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, reasons, mx = [], set(), None
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------
def oracle_step(sample_tokens, state):
    """One step of the oracle on the benchmark's workload: projection + quantise + pack of the four weight matrices of
    the layer (W + U), then the four GEMMs on the first `sample_tokens` tokens.  Returns (seconds, dense-equivalent ops,
    seconds of the pack part)."""
    import oracle
    import workloads as wl
    n, m, bits = PATTERN
    if "layer" not in state:
        oracle.set_threads(oracle.max_threads())
        rng = np.random.default_rng(2)
        state["layer"] = []
        for name, k, out in wl.BERT_LARGE_GEMMS:
            W = wl.normal(rng, (out, k), wl.W_STD)
            U = wl.normal(rng, (out, k), wl.U_STD)
            b = wl.normal(rng, (out,), wl.W_STD)
            state["layer"].append((W, U, b, wl.random_int8([5, k, out], (TOKENS, k))))
    t0 = time.perf_counter()
    packed = [oracle.project_pack(W, U, n, m, bits) for (W, U, b, X) in state["layer"]]
    t_pack = time.perf_counter() - t0
    ops = 0.0
    for (v, meta, s), (W, U, b, X) in zip(packed, state["layer"]):
        D = oracle.unpack(v, meta, W.shape[0], W.shape[1], n, m, bits)
        oracle.int_linear(X[:sample_tokens], D, 0.03, s, b, want_acc=False)
        ops += gemm_ops(sample_tokens, W.shape[1], W.shape[0])
    return time.perf_counter() - t0, ops, t_pack


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    state = {}
    sample_tokens = 512
    for _ in range(max(args.warmup, 1)):
        oracle_step(sample_tokens, state)
    secs, ops = 0.0, 0.0
    for _ in range(args.steps):
        s, o, _ = oracle_step(sample_tokens, state)
        secs += s
        ops += o
    value = ops / secs / 1e12
    cores = oracle.max_threads()
    sample = f"pack of the layer's four matrices + its four GEMMs on the first {sample_tokens} of 16384 tokens per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def cpu_baseline(budget_s=25.0):
    """The oracle, as it stands, on the host cores: the SAME step the GPU runs (four matrices packed, four GEMMs) on
    as many of the 16384 tokens as fit the budget (all of them on the usual 16 cores), and the projection/pack of the
    24-layer sweep (timed in full when it fits the budget, else one layer scaled by 24 and marked)."""
    import oracle
    import workloads as wl
    state = {}
    oracle_step(16, state)                       # builds the inputs
    probe, _, _ = oracle_step(64, state)
    _, _, t_pack = oracle_step(16, state)
    per_token = max(probe - t_pack, 1e-4) / 64
    tokens = int(max(64, min(TOKENS, (budget_s - t_pack) / per_token)))
    secs, ops, t_pack = oracle_step(tokens, state)
    full = tokens == TOKENS
    out = {"value": ops / secs / 1e12, "unit": "TOPS", "cores": oracle.max_threads(), "kind": "oracle",
           "seconds": secs, "pack_seconds": t_pack,
           "sample": (f"the whole step: pack of the layer's four matrices + its four GEMMs on all {TOKENS} tokens"
                      if full else f"pack of the layer's four matrices + its four GEMMs on the first {tokens} of "
                                   f"{TOKENS} tokens (GEMM time scales with the tokens: extrapolated to "
                                   f"{t_pack + (secs - t_pack) * TOKENS / tokens:.1f} s for the whole step)") + f" ({secs:.1f} s)"}
    # projection/pack sweep: 96 matrices, 302 M parameters, 2:4 / 8 bit
    n, m, bits = PATTERN
    shapes = wl.pack_sweep_shapes()
    layer_s = t_pack
    if layer_s * 24 <= budget_s:
        t0 = time.perf_counter()
        for i, (o, k) in enumerate(shapes):
            W, U = wl.pack_sweep_matrix(3, i % 4, o, k)   # the matrices' values do not change the oracle's work
            oracle.project_pack(W, U, n, m, bits)
        # drawing the inputs is not the method's work: time it separately and take it off
        t_all = time.perf_counter() - t0
        t0 = time.perf_counter()
        for i, (o, k) in enumerate(shapes):
            wl.pack_sweep_matrix(3, i % 4, o, k)
        t_draw = time.perf_counter() - t0
        out["pack_sweep"] = {"seconds": t_all - t_draw, "gbs": sum(pack_bytes(o, k, n, m, bits) for o, k in shapes) / (t_all - t_draw) / 1e9,
                             "extrapolated": False}
    else:
        out["pack_sweep"] = {"seconds": layer_s * 24, "gbs": sum(pack_bytes(o, k, n, m, bits) for o, k in shapes) / (layer_s * 24) / 1e9,
                             "extrapolated": True, "note": "one layer (4 of 96 matrices) timed, scaled by 24"}
    return out


def reduce_max_ms(ms, world, device="cpu"):
    """Time of the slowest rank (all ranks get it).  One scalar all-reduce; the data path has none."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ops_per_rank_step, world, ms_per_step):
    """Aggregate throughput of `world` ranks that each do the same per-GPU work (weak scaling)."""
    return world * ops_per_rank_step / (ms_per_step * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------
def source_hash():
    """Hash of the kernel sources: ties the DRAM-traffic figures under profiles/ to the kernels they were taken from."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2206_15014_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic():
    """DRAM bytes per launch from the ncu capture summarised in profiles/dram_traffic.txt ("key bytes" lines under a
    "sources <hash>" line).  Empty when the kernels have changed since the capture: the figures would be stale."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    out, ok = {}, False
    if os.path.exists(path):
        for line in open(path):
            f = line.split()
            if len(f) >= 2 and f[0] == "sources":
                ok = f[1] == source_hash()
            elif len(f) >= 2 and not line.startswith("#") and f[1].isdigit():
                out[f[0]] = int(f[1])
    return out if ok else {}


def gemm_entry(us, tokens, k, out, pk, n=2, m=4, bits=8, ybytes=4):
    """Time of one GEMM launch with its three roofline fractions: of the sparse INT8 tensor peak, of the HBM peak,
    and of the bound that applies, min(tensor, HBM) = the longer of the two ideal times."""
    ops, byt = gemm_ops(tokens, k, out), gemm_bytes(tokens, k, out, n, m, bits, ybytes)
    sparse_peak = 4.0 * pk["bf16_tflops"]
    t_tensor, t_hbm = ops / sparse_peak / 1e6, byt / pk["hbm_gbs"] / 1e3   # microseconds
    return {"us": us, "tops": ops / us / 1e6, "gbs": byt / us / 1e3,
            "frac_sparse_int8_peak_measured": ops / us / 1e6 / sparse_peak,
            "frac_sparse_int8_peak_nominal": ops / us / 1e6 / NOMINAL_SPARSE_INT8_TOPS,
            "frac_hbm_measured": byt / us / 1e3 / pk["hbm_gbs"],
            "frac_min_bound": max(t_tensor, t_hbm) / us, "bound": "tensor" if t_tensor > t_hbm else "hbm"}


def time_stream(torch, fn, iters, warm=20):
    """Average microseconds of fn() launched back to back `iters` times on the current stream."""
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


def packed_layer(nm, torch, dev, gemms, tokens, n, m, bits, seed, sets=4):
    """Device buffers of one encoder layer's GEMMs with weights projected and packed by the library: `sets` rotating
    X / Y buffer sets per GEMM (so that back-to-back launches really write to HBM), one packed weight each."""
    import workloads as wl
    rng = np.random.default_rng(seed)
    layer, status = [], torch.zeros(1, dtype=torch.int32, device=dev)
    for name, k, out in gemms:
        W = torch.from_numpy(wl.normal(rng, (out, k), wl.W_STD)).to(dev)
        b = torch.from_numpy(wl.normal(rng, (out,), wl.W_STD)).to(dev)
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        values = torch.empty(vb, dtype=torch.uint8, device=dev)
        meta = torch.empty(max(mb // 4, 1), dtype=torch.int32, device=dev)
        scales = torch.empty(out, dtype=torch.float32, device=dev)
        nm.nm_project_pack(W, None, out, k, n, m, bits, values, meta if mb else None, scales, status)
        X = [torch.from_numpy(wl.random_int8([5, k, out, i], (tokens, k))).to(dev) for i in range(sets)]
        Y = [torch.empty((tokens, out), dtype=torch.float32, device=dev) for _ in range(sets)]
        layer.append({"name": name, "k": k, "out": out, "b": b, "scales": scales, "X": X, "Y": Y,
                      "keep": (values, meta), "desc": nm.make_packed(out, k, n, m, bits, values, meta if mb else None)})
    assert nm.nm_poll_status(status) == nm.NM_OK
    return layer


def extra_configs(nm, torch, dev, pk, status):
    """Timed entries for the other workload configurations (each also a parity-test case): the single 128 x 768
    projection (a latency, in microseconds), the BERT-base layer at 4096 tokens, the BERT-large layer at 4096 tokens
    and with packed 4-bit codes at 16384 tokens, the 48-GEMM heterogeneous chain at 6144 tokens with its re-quantise
    steps, and the whole-model projection of the search (Sec. 4)."""
    import workloads as wl
    out = {}
    sx = 0.03
    # ---- configuration 1: one BERT-base attention output projection, 128 tokens: latency --------------------------
    lay = packed_layer(nm, torch, dev, (("attn_out", 768, 768),), 128, 2, 4, 8, seed=0)[0]
    call = lambda i: nm.nm_int_linear(lay["X"][i % 4], 128, lay["desc"], sx, lay["scales"], lay["b"], lay["Y"][i % 4], status=status)
    lat = []
    for i in range(60):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        call(i)
        torch.cuda.synchronize()
        lat.append((time.perf_counter() - t0) * 1e6)
    # the same launches replayed from a CUDA graph: what the device needs per launch without the host's share
    # (Python, ctypes and the launch call cost more than this kernel runs)
    graph_us = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(8):
                call(i)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(64):
                    call(i)
            torch.cuda.synchronize()
            graph_us = time_stream(torch, lambda i: g.replay(), 20, warm=3) / 64
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
    except Exception as e:   # a capture failure must not cost the benchmark line
        graph_us = None
        print("graph replay of the single projection failed: " + repr(e), file=sys.stderr)
    out["single_projection_128x768"] = {"latency_us_call_to_completion": float(np.median(lat[10:])),
                                        "us_back_to_back": time_stream(torch, call, 400),
                                        "us_back_to_back_from_a_graph": graph_us,
                                        "note": "all operands resident in L2: a latency figure, no roofline"}
    # ---- configurations 2 and 3: encoder-layer GEMMs, one launch after the other ------------------------------------
    for key, gemms, tokens, bits in (("bert_base_4096tok_int8", wl.BERT_BASE_GEMMS, 4096, 8),
                                     ("bert_large_4096tok_int8", wl.BERT_LARGE_GEMMS, 4096, 8),
                                     ("bert_large_16384tok_int4", wl.BERT_LARGE_GEMMS, 16384, 4)):
        layer = packed_layer(nm, torch, dev, gemms, tokens, 2, 4, bits, seed=1 if gemms is wl.BERT_BASE_GEMMS else 2)
        entry, total = {}, 0.0
        for g in layer:
            us = time_stream(torch, lambda i, g=g: nm.nm_int_linear(g["X"][i % 4], tokens, g["desc"], sx, g["scales"], g["b"],
                                                                     g["Y"][i % 4], status=status), 200)
            entry[g["name"]] = gemm_entry(us, tokens, g["k"], g["out"], pk, bits=bits)
            total += us
        def whole(i, layer=layer):
            for g in layer:
                nm.nm_int_linear(g["X"][i % 4], tokens, g["desc"], sx, g["scales"], g["b"], g["Y"][i % 4], status=status)
        entry["layer_us"] = time_stream(torch, whole, 100)
        entry["layer_tops"] = sum(gemm_ops(tokens, g["k"], g["out"]) for g in layer) / entry["layer_us"] / 1e6
        out[key] = entry
        del layer
        torch.cuda.empty_cache()
    # ---- configuration 5: heterogeneous 12-layer chain, 6144 tokens, re-quantised between GEMMs ------------------------
    T, hidden = 6144, 768
    modes, h0, weights = wl.chain_case(4, layers=12, tokens=T)
    chain = []
    for layer_modes, wrow in zip(modes, weights):
        for mode, (W, b) in zip(layer_modes, wrow):
            n, m, bits = wl.CHAIN_MODES[mode]
            o, k = W.shape
            vb, mb = nm.nm_packed_sizes(o, k, n, m, bits)
            values = torch.empty(vb, dtype=torch.uint8, device=dev)
            meta = torch.empty(max(mb // 4, 1), dtype=torch.int32, device=dev)
            scales = torch.empty(o, dtype=torch.float32, device=dev)
            nm.nm_project_pack(torch.from_numpy(W).to(dev), None, o, k, n, m, bits, values, meta if mb else None, scales, status)
            chain.append({"out": o, "k": k, "b": torch.from_numpy(b).to(dev), "scales": scales, "keep": (values, meta),
                          "desc": nm.make_packed(o, k, n, m, bits, values, meta if mb else None), "mode": (n, m, bits)})
    Ybuf = torch.empty((T, 3072), dtype=torch.float32, device=dev)      # widest output
    Vbuf = torch.empty((T, hidden), dtype=torch.float32, device=dev)
    Xbuf = [torch.empty((T, 3072), dtype=torch.int8, device=dev) for _ in range(2)]
    amax = torch.zeros(2, dtype=torch.float32, device=dev)
    sxd = torch.empty(2, dtype=torch.float32, device=dev)
    H0 = torch.from_numpy(h0).to(dev)

    def run_chain(_):
        amax.zero_()
        nm.nm_absmax(H0, H0.numel(), amax[0:1])
        nm.nm_quantize_act(H0, H0.numel(), amax[0:1], Xbuf[0], sxd[0:1])
        cur = 0
        for i, g in enumerate(chain):
            o, k = g["out"], g["k"]
            Y = Ybuf.view(-1)[: T * o].view(T, o)
            X = Xbuf[cur].view(-1)[: T * k].view(T, k)
            nxt = cur ^ 1
            amax[nxt:nxt + 1].zero_()
            if i % 4 == 0:   # QKV: only the V slice feeds the next GEMM (a copy, no arithmetic), then its own maximum
                nm.nm_int_linear_dsx(X, T, g["desc"], sxd[cur:cur + 1], g["scales"], g["b"], Y, None, status=status)
                Vbuf.copy_(Y[:, 2 * hidden:])
                nm.nm_absmax(Vbuf, Vbuf.numel(), amax[nxt:nxt + 1])
                src, cnt = Vbuf, Vbuf.numel()
            else:            # the GEMM's own running max|Y| feeds the quantiser
                nm.nm_int_linear_dsx(X, T, g["desc"], sxd[cur:cur + 1], g["scales"], g["b"], Y, amax[nxt:nxt + 1], status=status)
                src, cnt = Y, Y.numel()
            nm.nm_quantize_act(src, cnt, amax[nxt:nxt + 1], Xbuf[nxt], sxd[nxt:nxt + 1])
            cur = nxt

    chain_us = time_stream(torch, run_chain, 20, warm=3)
    chain_ops = sum(gemm_ops(T, g["k"], g["out"]) for g in chain)
    out["hetero_chain_48gemm_6144tok"] = {
        "us": chain_us, "tops_dense_equivalent": chain_ops / chain_us / 1e6, "gemms": len(chain),
        "modes": {f"{n}:{m}/{b}b": int(sum(1 for g in chain if g["mode"] == (n, m, b))) for (n, m, b) in wl.CHAIN_MODES},
        "note": "48 GEMM launches + 48 re-quantise launches (+ 12 slice copies and 13 absmax launches), device-resident scales"}
    del chain, Ybuf, Vbuf, Xbuf
    torch.cuda.empty_cache()
    # ---- search support: a whole BERT-base encoder stack projected to a heterogeneous configuration in one call ---------
    cfgs = {"Q4": (4, 4, 4), "Q8": (4, 4, 8), "S4": (2, 4, 4), "S8": (2, 4, 8)}
    row = ["S8", "S8", "Q8", "Q4", "S4", "S4"]       # one Table-4-style row: Q, K, V, attention output, FFN1, FFN2
    shapes6 = [(768, 768)] * 4 + [(3072, 768), (768, 3072)]
    gen = torch.Generator(device=dev)
    gen.manual_seed(6)
    jobs, nbytes = [], 0.0
    for layer in range(12):
        for comp, (o, k) in enumerate(shapes6):
            n, m, bits = cfgs[row[(comp + layer) % 6]]   # the components' formats rotate from layer to layer
            W = torch.empty((o, k), dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
            vb, mb = nm.nm_packed_sizes(o, k, n, m, bits)
            jobs.append((W, None, n, m, bits, torch.empty(vb, dtype=torch.uint8, device=dev),
                         torch.empty(max(mb // 4, 1), dtype=torch.int32, device=dev) if mb else None,
                         torch.empty(o, dtype=torch.float32, device=dev)))
            nbytes += pack_bytes(o, k, n, m, bits, with_u=False)
    arr = nm.make_pack_jobs(jobs)
    ws_bytes = nm.nm_pack_workspace_bytes(len(jobs))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    us = time_stream(torch, lambda i: nm.nm_project_pack_batched(arr, len(jobs), ws, ws_bytes, status), 50, warm=5)
    out["whole_model_projection_bert_base"] = {
        "us_per_configuration": us, "matrices": len(jobs), "gbs": nbytes / us / 1e3,
        "frac_hbm_measured": nbytes / us / 1e3 / pk["hbm_gbs"],
        "seconds_for_905_configurations": 905 * us / 1e6,
        "note": "72 matrices (85 M parameters, 340 MB: larger than L2), four formats rotating over the components, one call"}
    return out


def ffn1_stream_probe(nm, torch, dev, d, tokens, status):
    """The resident-weight pair kernel's traffic on one GEMM without its arithmetic (nm_probe_tma_stream): X loads
    through the ring + Y stores, and Y stores alone.  Times from the CTAs' own globaltimer stamps, median of three."""
    import numpy as np
    clocks = torch.zeros((torch.cuda.get_device_properties(dev).multi_processor_count, 4), dtype=torch.int64, device=dev)
    out, k = d["out"], d["k"]
    res = {}
    for name, loads, stores in (("loads_and_stores_us", 2, 1), ("stores_only_us", 0, 1)):
        spans = []
        for _ in range(4):
            ctas = nm.nm_probe_tma_stream(d["values"], out, k // 2, d["X"], tokens, k, d["Y"], 128, 128, 96, 2, 5, 0, 1, 0,
                                          loads, stores, 1, 0, clocks, None, status)
            torch.cuda.synchronize()
            c = clocks[:ctas].cpu().numpy()
            spans.append(float(c[:, 3].max() - c[:, 2].min()) / 1e3)
        res[name] = float(np.median(spans[1:]))
    ybytes = tokens * out * 4
    res["stores_only_gbs"] = ybytes / res["stores_only_us"] / 1e3
    return res


def run_cuda(args):
    TOKENS = args.tokens
    PATTERN = (2, 4, args.bits)
    import torch
    import torch.distributed as dist
    import workloads as wl
    import paper_2206_15014_b200 as nm

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    for kv in args.option:   # A/B runs of a kernel choice; recorded in the line's config
        k, v = kv.split("=")
        nm.nm_debug_set_option(k, int(v))   # raises on an unknown name
    n, m, bits = PATTERN
    pk = peaks()
    YDTYPE = {"f32": torch.float32, "int8": torch.int8, "bf16": torch.bfloat16}[args.out]
    YB = {"f32": 4, "int8": 1, "bf16": 2}[args.out]

    # ---- inputs (seeded per rank: independent batches, weak scaling) ---------------------------
    rng = np.random.default_rng([2, rank])
    layer = []
    for name, k, out in wl.BERT_LARGE_GEMMS:
        W = wl.normal(rng, (out, k), wl.W_STD)
        U = wl.normal(rng, (out, k), wl.U_STD)
        b = wl.normal(rng, (out,), wl.W_STD)
        Xq = wl.random_int8([5, rank, k, out], (TOKENS, k))
        layer.append((name, k, out, W, U, b, Xq))

    host = []  # pinned host copies for the end-to-end leg: inputs, and every result of the step
    devbuf = []
    for name, k, out, W, U, b, Xq in layer:
        hW, hU, hX = (torch.from_numpy(a).pin_memory() for a in (W, U, Xq))
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        d = {"W": hW.to(dev), "U": hU.to(dev), "X": hX.to(dev), "b": torch.from_numpy(b).to(dev),
             "values": torch.empty(vb, dtype=torch.uint8, device=dev),
             "meta": torch.empty(mb // 4, dtype=torch.int32, device=dev),
             "scales": torch.empty(out, dtype=torch.float32, device=dev),
             "Y": torch.empty((TOKENS, out), dtype=YDTYPE, device=dev), "k": k, "out": out, "name": name}
        d["desc"] = nm.make_packed(out, k, n, m, bits, d["values"], d["meta"])
        hres = {key: torch.empty(d[key].shape, dtype=d[key].dtype).pin_memory() for key in ("Y", "values", "meta", "scales")}
        host.append((hW, hU, hX, hres))
        devbuf.append(d)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    jobs = nm.make_pack_jobs([(d["W"], d["U"], n, m, bits, d["values"], d["meta"], d["scales"]) for d in devbuf])
    ws_bytes = nm.nm_pack_workspace_bytes(len(devbuf))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    sx = 0.03
    SY = 0.05  # static output scale of the int8-output variant (outputs are ~N(0, 0.5): little clamping)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    kernel_events = {"pack": []}
    for d in devbuf:
        kernel_events[d["name"]] = []

    def linear(d):
        if args.out == "f32":
            nm.nm_int_linear(d["X"], TOKENS, d["desc"], sx, d["scales"], d["b"], d["Y"], status=status)
        elif args.out == "int8":
            nm.nm_int_linear_q8(d["X"], TOKENS, d["desc"], sx, d["scales"], d["b"], SY, d["Y"], status=status)
        else:
            nm.nm_int_linear_bf16(d["X"], TOKENS, d["desc"], sx, d["scales"], d["b"], d["Y"], status=status)

    names = ["pack"] + [d["name"] for d in devbuf]

    def step(record=None):
        """One step.  record = the name of ONE launch to put an event pair around (the other four stay chained)."""
        for name in names:
            if name == record:
                e0, e1 = ev(), ev()
                e0.record()
            if name == "pack":
                nm.nm_project_pack_batched(jobs, len(devbuf), ws, ws_bytes, status)
            else:
                linear(next(d for d in devbuf if d["name"] == name))
            if name == record:
                e1.record()
                kernel_events[name].append((e0, e1))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return reduce_max_ms(ms, world, dev)

    # ---- headline: device-resident timing, nothing but the step's five launches in the timed region ------------------
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    # the device has just idled for a quarter of a second while the clock sampler started, and the first launches after
    # an idle spell are slow (120 us in all: 6 us per step of a 20-step run).  Untimed steps bring it back to the state
    # a long run has; the timed region follows without a pause.
    SPIN_UP = 50
    for _ in range(SPIN_UP):
        step()
    barrier()
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    barrier()
    ms = max_over_ranks(t0.elapsed_time(t1))
    rc = nm.nm_poll_status(status)
    if rc != nm.NM_OK:
        raise RuntimeError("device status: " + nm.nm_strerror(rc))
    ms_per_step = ms / args.steps
    ops_step = sum(gemm_ops(TOKENS, d["k"], d["out"]) for d in devbuf)
    value = whole_job_tops(ops_step, world, ms_per_step)

    # ---- the same steps once more, each with an event pair around ONE of its five launches in turn: the per-kernel
    # breakdown.  (An event between two launches keeps the second from starting its set-up during the first one's tail,
    # so a bracketed launch reads a little longer than it takes inside the headline region.) ----
    prof_steps = 5 * max(8, min(args.steps // 5, 40))
    p0, p1 = ev(), ev()
    p0.record()
    for j in range(prof_steps):
        step(record=names[j % 5])
    p1.record()
    barrier()
    profiled_ms_per_step = p0.elapsed_time(p1) / prof_steps
    kern = {}
    for name, pairs in kernel_events.items():
        kern[name] = float(np.mean([a.elapsed_time(b) for a, b in pairs])) * 1e3  # microseconds

    # ---- end to end: pinned host buffers in, every result of the step out (Y and the packed weights), every step --------
    # Copies run on their own streams: the inputs of step i + 1 go in (after step i's kernels have read the
    # old ones) while the outputs of step i are still leaving; the kernels of step i + 1 wait for both.
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in, ev_comp, ev_out = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()

    def e2e_step():
        s_in.wait_event(ev_comp)
        with torch.cuda.stream(s_in):
            for (hW, hU, hX, hres), d in zip(host, devbuf):
                d["W"].copy_(hW, non_blocking=True)
                d["U"].copy_(hU, non_blocking=True)
                d["X"].copy_(hX, non_blocking=True)
            ev_in.record(s_in)
        main.wait_event(ev_in)
        main.wait_event(ev_out)
        step()
        ev_comp.record(main)
        s_out.wait_event(ev_comp)
        with torch.cuda.stream(s_out):
            for (hW, hU, hX, hres), d in zip(host, devbuf):
                for key, h in hres.items():
                    h.copy_(d[key], non_blocking=True)
            ev_out.record(s_out)

    e2e_steps = max(3, min(args.steps, 20))
    e2e_step()
    main.wait_event(ev_out)
    barrier()
    t0.record()
    for _ in range(e2e_steps):
        e2e_step()
    main.wait_event(ev_out)  # the last step's outputs have reached the host
    t1.record()
    barrier()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1)) / e2e_steps
    h2d = sum(hW.numel() * 4 + hU.numel() * 4 + hX.numel() for hW, hU, hX, hres in host)
    d2h = sum(h.numel() * h.element_size() for hW, hU, hX, hres in host for h in hres.values())
    clocks = sampler.stop() if rank == 0 else None

    # ---- projection/pack on the full 24-layer sweep (its own roofline), rank 0 only ---------------
    pack_info = None
    if rank == 0 and not args.skip_sweep:
        pack_info = pack_sweep(nm, torch, dev, status)
    # ---- the dominant GEMMs launched alone, back to back over rotating buffers; write-only bandwidth of the device ------
    alone = {}
    stream_probe = None
    if rank == 0:
        for d in devbuf:
            Ys = [d["Y"]] + [torch.empty_like(d["Y"]) for _ in range(2)]
            def one(i, d=d, Ys=Ys):
                saved, d["Y"] = d["Y"], Ys[i % 3]
                linear(d)
                d["Y"] = saved
            alone[d["name"]] = time_stream(torch, one, 100)
            del Ys
        # the projection launched alone: two more copies of W and U, so that no launch finds its inputs in L2
        sets = [jobs]
        extra = []
        for _ in range(2):
            cp = [(d["W"].clone(), d["U"].clone()) for d in devbuf]
            extra.append(cp)
            sets.append(nm.make_pack_jobs([(W, U, n, m, bits, d["values"], d["meta"], d["scales"]) for (W, U), d in zip(cp, devbuf)]))
        alone["pack"] = time_stream(torch, lambda i: nm.nm_project_pack_batched(sets[i % 3], len(devbuf), ws, ws_bytes, status), 100)
        del sets, extra
        # what FFN1's byte stream costs with no arithmetic: the library's traffic probe walks the same tiles in the same
        # order with the same TMA operations (X through a five-stage ring, Y in [16 tokens][32 channels] boxes) --
        # stores alone, and loads + stores.  fp32 outputs and 8-bit weights only (the probe's tile is that kernel's).
        if args.out == "f32" and bits == 8:
            stream_probe = ffn1_stream_probe(nm, torch, dev, next(d for d in devbuf if d["name"] == "ffn1"), TOKENS, status)
        torch.cuda.empty_cache()
    extras = None
    if rank == 0 and not args.skip_configs and TOKENS == 16384 and bits == 8 and args.out == "f32":
        for d in devbuf:   # make room: the extra configurations bring their own buffers
            d.pop("W"); d.pop("U")
        torch.cuda.empty_cache()
        extras = extra_configs(nm, torch, dev, pk, status)
        rc = nm.nm_poll_status(status)
        if rc != nm.NM_OK:
            raise RuntimeError("device status in the extra configurations: " + nm.nm_strerror(rc))

    if rank == 0:
        sparse_peak = 4.0 * pk["bf16_tflops"]
        traffic = recorded_traffic()
        full_size = TOKENS == 16384 and bits == 8 and args.out == "f32"
        per_kernel = {}
        for d in devbuf:
            e = gemm_entry(kern[d["name"]], TOKENS, d["k"], d["out"], pk, n, m, bits, YB)
            e["us_launched_alone"] = alone[d["name"]]
            per_kernel[d["name"]] = e
        pbytes = sum(pack_bytes(d["out"], d["k"], n, m, bits) for d in devbuf)
        # in the step the launch follows FFN2 and FFN1, whose last outputs are still dirty in L2 and are written back
        # while it reads; launched alone (inputs rotating, never in L2) it only moves its own bytes
        per_kernel["pack_layer"] = {"us": kern["pack"], "gbs": pbytes / kern["pack"] / 1e3,
                                    "frac_hbm_measured": pbytes / kern["pack"] / 1e3 / pk["hbm_gbs"],
                                    "us_launched_alone": alone["pack"],
                                    "frac_hbm_launched_alone": pbytes / alone["pack"] / 1e3 / pk["hbm_gbs"]}
        if pack_info:
            per_kernel["pack_sweep"] = pack_info
        # dominant kernel of the step: the FFN1 GEMM launch (longest).  Its bytes are 93 % fp32 Y written in tiles of
        # 128 channels x 192 tokens; `stream_probe` says what that byte stream costs on this device with no arithmetic
        # (`frac_of_stream_probe` = probe time / kernel time launched alone).  `traffic` = dram__bytes_read.sum + dram__bytes_write.sum of one launch at this size
        # (ncu; part of Y is still in the 126 MB L2 when the kernel ends, hence below the algorithmic bytes).
        dom = per_kernel["ffn1"]
        k1 = f"nm_gemm_pair_kernel<sparse,192,{args.out},resident" + (">" if bits == 8 else ",builder warps>")
        k2 = f"nm_gemm_wide_kernel<224,{args.out}" + (">" if bits == 8 else ",packed 4-bit codes>")
        roofline = {"kernel": k1 + " on ffn1 1024->4096", "bound": "hbm",
                    "achieved": dom["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": dom["gbs"] / pk["hbm_gbs"], "traffic": traffic.get("ffn1") if full_size else None,
                    "algorithmic_bytes": gemm_bytes(TOKENS, 1024, 4096, n, m, bits, YB), "peak_source": pk["source"],
                    "stream_probe": stream_probe,
                    "frac_of_stream_probe": (stream_probe["loads_and_stores_us"] / alone["ffn1"]) if stream_probe else None}
        f2 = per_kernel["ffn2"]
        roofline_tensor = {"kernel": k2 + " on ffn2 4096->1024", "bound": "tensor",
                           "achieved": f2["tops"], "peak": sparse_peak, "unit": "TOP/s",
                           "frac": f2["tops"] / sparse_peak,
                           "peak_note": "4 x measured bf16 burst (nominal int8-sparse : bf16-dense ratio)",
                           "frac_of_nominal_9000": f2["tops"] / NOMINAL_SPARSE_INT8_TOPS,
                           "frac_launched_alone": gemm_ops(TOKENS, 4096, 1024) / alone["ffn2"] / 1e6 / sparse_peak,
                           "frac_min_bound": f2["frac_min_bound"],
                           "traffic": traffic.get("ffn2") if full_size else None}
        line = {"metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
                "config": {"workload": WORKLOAD if TOKENS == 16384 else WORKLOAD + f" (reduced to {TOKENS} tokens)", "tokens": TOKENS, "pattern": "2:4", "bits": bits, "out": args.out,
                           "l2": "inputs+outputs per step (715 MB) exceed L2; no flush needed",
                           "spin_up_steps": SPIN_UP,
                           **({"options": list(args.option)} if args.option else {})},
                "clocks": clocks,
                "e2e": {"value": whole_job_tops(ops_step, world, e2e_ms), "unit": "TOPS",
                        "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
                "gpu_launches": 5 * args.steps,
                "profiled_pass": {"steps": prof_steps, "ms_per_step": profiled_ms_per_step,
                                  "note": "per-kernel times come from this separate pass: every step has an event pair around one of its five launches"},
                "roofline": roofline, "roofline_tensor": roofline_tensor, "kernels": per_kernel}
        if extras:
            line["configs"] = extras
        if pack_info:
            line["roofline_pack"] = {"kernel": "pack_kernel<2,4,8> on the 24-layer sweep", "bound": "hbm",
                                     "achieved": pack_info["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                                     "frac": pack_info["gbs"] / pk["hbm_gbs"],
                                     "frac_of_nominal_8000": pack_info["gbs"] / NOMINAL_HBM_GBS, "traffic": traffic.get("pack_sweep"),
                                     "algorithmic_bytes": pack_info["bytes"]}
            adm = pack_info["admm_step_2:4/8b"]
            line["roofline_admm"] = {"kernel": "pack_kernel<2,4,8,dense outputs> (ADMM step: Z and U_next) on the 24-layer sweep",
                                     "bound": "hbm", "achieved": adm["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                                     "frac": adm["gbs"] / pk["hbm_gbs"], "traffic": traffic.get("admm_sweep"),
                                     "algorithmic_bytes": adm["bytes"]}
        line["cpu_baseline"] = cpu_baseline() if (world == 1 and not args.skip_cpu) else None
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def pack_sweep(nm, torch, dev, status, reps=5):
    """Projection/pack of all 96 BERT-large encoder weights (302 M parameters, 2.4 GB of fp32 W+U)
    in one batched launch, for every (n:m, bits) of the sweep; returns time and algorithmic GB/s of the
    2:4 / 8-bit variant plus a per-variant table."""
    import workloads as wl
    shapes = wl.pack_sweep_shapes()
    gen = torch.Generator(device=dev)
    gen.manual_seed(3)
    mats = []
    for out, k in shapes:
        W = torch.empty((out, k), dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
        U = torch.empty((out, k), dtype=torch.float32, device=dev).normal_(0.0, 0.002, generator=gen)
        sizes = [nm.nm_packed_sizes(out, k, n, m, bits) for (n, m, bits) in wl.PACK_SWEEP]
        vb, mb = max(v for v, _ in sizes), max(x for _, x in sizes)  # buffers large enough for every variant
        mats.append((W, U, torch.empty(vb, dtype=torch.uint8, device=dev), torch.empty(mb // 4, dtype=torch.int32, device=dev),
                     torch.empty(out, dtype=torch.float32, device=dev)))
    ws_bytes = nm.nm_pack_workspace_bytes(len(mats))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    table = {}
    for (n, m, bits) in wl.PACK_SWEEP:
        arr = nm.make_pack_jobs([(W, U, n, m, bits, v, mt, sc) for (W, U, v, mt, sc) in mats])
        nbytes = sum(pack_bytes(o, k, n, m, bits) for o, k in shapes)
        for _ in range(3):
            nm.nm_project_pack_batched(arr, len(mats), ws, ws_bytes, status)
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            nm.nm_project_pack_batched(arr, len(mats), ws, ws_bytes, status)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        us = float(np.median(times)) * 1e3
        table[f"{n}:{m}/{bits}b"] = {"us": us, "gbs": nbytes / us / 1e3, "bytes": nbytes}
    # group-wise scales (32 output channels per scale, the paper's default), one batched call: two passes over
    # W and U (row maxima per group, then the projection); GB/s on the same algorithmic bytes as the per-channel pack
    grouped_jobs = nm.make_pack_jobs([(W, U, 2, 4, 8, v, mt, sc) for (W, U, v, mt, sc) in mats])
    def grouped_pass():
        nm.nm_project_pack_grouped_batched(grouped_jobs, len(mats), 32, ws, ws_bytes, status)
    grouped_pass()
    torch.cuda.synchronize()
    times = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        grouped_pass()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    grouped_us = float(np.median(times)) * 1e3
    grouped = {"us": grouped_us, "gbs": table["2:4/8b"]["bytes"] / grouped_us / 1e3, "bytes": table["2:4/8b"]["bytes"],
               "launches": 4, "group_rows": 32}
    # ADMM-Dist scale search (32 candidate scales per output channel) followed by the projection at the chosen
    # scale, 2:4 with 4-bit and 8-bit codes, one batched call (2 launches).  The search is bound by instruction
    # issue, not by memory: reported as time and as candidate evaluations (kept value x candidate) per second.
    dist = {}
    kept = sum(o * k for o, k in shapes) // 2
    for bits in (4, 8):
        dist_jobs = nm.make_pack_jobs([(W, U, 2, 4, bits, v, mt, sc) for (W, U, v, mt, sc) in mats])
        def dist_pass():
            nm.nm_project_pack_dist_batched(dist_jobs, len(mats), 32, ws, ws_bytes, status)
        dist_pass()
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dist_pass()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        us = float(np.median(times)) * 1e3
        dist[f"2:4/{bits}b"] = {"us": us, "search_us": us - table[f"2:4/{bits}b"]["us"], "candidates": 32, "launches": 2,
                                "evals_per_s": kept * 32 / (us - table[f"2:4/{bits}b"]["us"]) * 1e6}
    # ADMM step with dense outputs over the same 96 matrices (one batched call): W and U read, Z and
    # U_next (in place over U, so it runs last) written, 16 bytes per parameter; 2:4 / 8-bit, no packed outputs
    Zs = [torch.empty_like(W) for (W, U, v, mt, sc) in mats]
    admm_jobs = nm.make_admm_jobs([(W, U, 2, 4, 8, Z, U, None, None, None) for (W, U, v, mt, sc), Z in zip(mats, Zs)])
    admm_ws_bytes = nm.nm_admm_workspace_bytes(len(mats))
    admm_ws = torch.empty(admm_ws_bytes, dtype=torch.uint8, device=dev)
    def admm_pass():
        nm.nm_admm_project_batched(admm_jobs, len(mats), admm_ws, admm_ws_bytes, status)
    admm_pass()
    torch.cuda.synchronize()
    times = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        admm_pass()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    admm_us = float(np.median(times)) * 1e3
    admm_bytes = 16.0 * sum(o * k for o, k in shapes)
    head = table["2:4/8b"]
    return {"us": head["us"], "gbs": head["gbs"], "params": int(sum(o * k for o, k in shapes)),
            "bytes": head["bytes"], "matrices": len(shapes), "launches": 1, "variants": table,
            "grouped_2:4/8b": grouped, "admm_dist": dist,
            "admm_step_2:4/8b": {"us": admm_us, "gbs": admm_bytes / admm_us / 1e3, "bytes": admm_bytes, "launches": 1}}


def dist_case(bits):
    """A small ADMM-Dist case for profiler captures: eight 4096x1024 matrices (268 MB of W and U, larger than
    L2), 2:4, 32 candidates, one batched call = one search launch + one projection launch.  Prints its time."""
    import torch
    import paper_2206_15014_b200 as nm
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(3)
    mats = []
    for _ in range(8):
        out, k = 4096, 1024
        W = torch.empty((out, k), dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
        U = torch.empty((out, k), dtype=torch.float32, device=dev).normal_(0.0, 0.002, generator=gen)
        vb, mb = nm.nm_packed_sizes(out, k, 2, 4, bits)
        mats.append((W, U, 2, 4, bits, torch.empty(vb, dtype=torch.uint8, device=dev),
                     torch.empty(mb // 4, dtype=torch.int32, device=dev), torch.empty(out, dtype=torch.float32, device=dev)))
    ws_bytes = nm.nm_pack_workspace_bytes(len(mats))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    jobs = nm.make_pack_jobs(mats)
    for _ in range(3):
        nm.nm_project_pack_dist_batched(jobs, len(mats), 32, ws, ws_bytes, status)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    nm.nm_project_pack_dist_batched(jobs, len(mats), 32, ws, ws_bytes, status)
    e1.record()
    torch.cuda.synchronize()
    rc = nm.nm_poll_status(status)
    print(json.dumps({"case": "admm_dist 8 x [4096,1024] 2:4", "bits": bits, "candidates": 32,
                      "us": e0.elapsed_time(e1) * 1e3, "status": rc}))
    return 0 if rc == 0 else 1


def tma_probe(args):
    """Ceiling of the memory system for the pair GEMM's tile shapes: the kernel's TMA boxes, tile walk and stage
    ring with no arithmetic (nm_probe_tma_stream).  One JSON line per case: chip TB/s from CUDA events, bytes per
    clock per SM from the CTAs' own clock64 counters."""
    import torch
    import paper_2206_15014_b200 as nm
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    clocks = torch.zeros((torch.cuda.get_device_properties(dev).multi_processor_count, 4), dtype=torch.int64, device=dev)

    def case(name, out, k, tokens, a_rows, a_row_bytes, b_rows, b_slices, stages, band=0, repeat=1, delay=0, loads=3,
             stores=1, producers=1):
        w_row_bytes = k // 2                       # 2:4 int8 codes
        W = torch.randint(0, 255, (out, w_row_bytes), dtype=torch.uint8, device=dev)
        X = torch.randint(0, 255, (tokens, k), dtype=torch.uint8, device=dev)
        Y = torch.empty((tokens, out), dtype=torch.float32, device=dev)
        spans, cycles, ctas = [], [], 0
        for _ in range(4):   # the first run warms up; each run is timed by the CTAs' own clocks (launched on an idle
            ctas = nm.nm_probe_tma_stream(W, out, w_row_bytes, X, tokens, k, Y, a_rows, a_row_bytes, b_rows, b_slices,
                                          stages, band, repeat, delay, loads, stores, producers, 0, clocks, None, status)
            torch.cuda.synchronize()   # GPU, an event pair would also count the host's launch latency)
            c = clocks[:ctas].cpu().numpy()
            spans.append(float(c[:, 3].max() - c[:, 2].min()) / 1e3)
            cycles.append(float(np.median(c[:, 1] - c[:, 0])))
        rc = nm.nm_poll_status(status)
        us, cyc = float(np.median(spans[1:])), float(np.median(cycles[1:]))
        n_out_tiles, n_tok_tiles = -(-out // (2 * a_rows)), -(-tokens // (2 * b_rows))
        tiles = n_out_tiles * n_tok_tiles * repeat
        kblocks = w_row_bytes // a_row_bytes
        ld = tiles * kblocks * 2 * (((loads & 1) and a_rows * a_row_bytes) + ((loads & 2) and b_rows * 128 * b_slices))
        st = tiles * 2 * a_rows * 2 * b_rows * 4 if stores else 0
        print(json.dumps({"case": name, "status": rc, "span_us": round(us, 2), "tile": [2 * a_rows, 2 * b_rows],
                          "stage_bytes": a_rows * a_row_bytes + b_rows * 128 * b_slices, "stages": stages, "producers": producers,
                          "delay": delay, "loads": loads, "stores": stores, "repeat": repeat,
                          "load_MB": round(ld / 1e6, 1), "store_MB": round(st / 1e6, 1), "TBps": round((ld + st) / us / 1e6, 2),
                          "B_per_clk_per_SM": round((ld + st) / ctas / cyc, 1),
                          "clk_per_stage": round(cyc / (tiles * kblocks / (ctas / 2)), 1),
                          "sm_ghz": round(cyc / (us * 1e3), 3)}), flush=True)

    T, K, OUT = args.tokens, 4096, 1024
    # the streamed pair kernel's tile on FFN2 (256 channels x 192 tokens, 256 reduction elements per stage, five stages)
    for producers in (1, 2):
        for stores in (1, 0):
            case("ffn2 pair tile 256x192", OUT, K, T, 128, 128, 96, 2, 5, stores=stores, producers=producers)
    case("ffn2 pair tile 256x192, stage held 384 clk", OUT, K, T, 128, 128, 96, 2, 5, delay=384, producers=2)
    case("ffn2 pair tile 256x192, weights only", OUT, K, T, 128, 128, 96, 2, 5, loads=1, stores=0)
    case("ffn2 pair tile 256x192, X only", OUT, K, T, 128, 128, 96, 2, 5, loads=2, stores=0)
    for stages in (3, 4):
        case("ffn2 pair tile 256x192", OUT, K, T, 128, 128, 96, 2, stages, producers=2)
    # 128 reduction elements per stage: twice the stages of half the size
    case("ffn2 pair tile 256x192, 20 KB stages", OUT, K, T, 128, 64, 96, 1, 9, producers=2)
    # wider tiles: 512 channels per pair
    for b_rows in (96, 112, 128):
        for producers in (1, 2):
            for stores in (1, 0):
                case(f"ffn2 pair tile 512x{2 * b_rows}", OUT, K, T, 256, 64, b_rows, 1, 6 if b_rows < 128 else 5, stores=stores,
                     producers=producers)
    case("ffn2 pair tile 512x224, stage held 448 clk", OUT, K, T, 256, 64, 112, 1, 6, delay=448, producers=2)
    case("ffn2 pair tile 512x224, 4 stages", OUT, K, T, 256, 64, 112, 1, 4, producers=2)
    # stores alone (the producer arms its stages without loading anything): [16 tokens][32 channels] boxes as in the GEMMs,
    # then 8 KB boxes 32, 64 and 128 channels wide
    for stores in (1, 32, 64, 128):
        case("stores only, 512x256 tiles", OUT, K, T, 256, 64, 128, 1, 5, loads=0, stores=stores)
    # FFN1 (1024 -> 4096), where the weights stay in shared memory: the ring carries X only and Y is four times as large
    for loads, stores in ((2, 1), (2, 0), (0, 1)):
        case("ffn1 resident-weight tile 256x192 (X loads only)", 4096, 1024, T, 128, 128, 96, 2, 5, loads=loads, stores=stores)
    case("ffn1 resident-weight tile 256x192, stage held 640 clk", 4096, 1024, T, 128, 128, 96, 2, 5, loads=2, delay=640)
    # everything resident in L2: a small problem walked five times
    case("L2-resident 256x192", OUT, K, 19 * 192, 128, 128, 96, 2, 5, repeat=5, stores=0, producers=2)
    case("L2-resident 512x224", OUT, K, 37 * 224, 256, 64, 112, 1, 6, repeat=5, stores=0, producers=2)
    return 0


def trace_gemm(args):
    """Role-by-role time stamps of one GEMM launch from the library built with -DNM_TRACE (build.py --variant trace;
    run as NMSPARSE_LIB=paper_2206_15014_b200/libnmsparse_trace.so python bench.py --trace-gemm TOKENS,K,OUT).  CTA 0
    stamps clock64() per pipeline stage (producer got the stage / issued its loads, gate saw it full, MMA thread was
    handed it / had issued its MMAs) and per tile (accumulators full, epilogue done).  Prints one JSON line of medians
    and the per-tile rows; the launch itself is the product's kernel with the stamps added."""
    import torch
    import paper_2206_15014_b200 as nm
    dev = torch.device("cuda:0")
    T, K, OUT = (int(x) for x in args.trace_gemm.split(","))
    for kv in args.option:
        k, v = kv.split("=")
        nm.nm_debug_set_option(k, int(v))
    X = torch.randint(-127, 127, (T, K), dtype=torch.int8, device=dev)
    vals = torch.randint(-127, 127, (OUT, K // 2 * args.bits // 8), dtype=torch.int8, device=dev)   # 8-bit or packed 4-bit codes
    meta = torch.full((OUT, K // 32), 0x4E4E4E4E, dtype=torch.int32, device=dev)   # valid 2:4 positions (2,3) and (0,1)
    sw, b = torch.ones(OUT, device=dev), torch.zeros(OUT, device=dev)
    Y = torch.empty((T, OUT), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    desc = nm.make_packed(OUT, K, 2, 4, args.bits, vals, meta)
    trace = torch.zeros((576, 8), dtype=torch.int64, device=dev)
    if args.out == "int8":
        Y = torch.empty((T, OUT), dtype=torch.int8, device=dev)
        run = lambda: nm.nm_int_linear_q8(X, T, desc, 0.01, sw, b, 0.05, Y, status=status)
    elif args.out == "bf16":
        Y = torch.empty((T, OUT), dtype=torch.bfloat16, device=dev)
        run = lambda: nm.nm_int_linear_bf16(X, T, desc, 0.01, sw, b, Y, status=status)
    else:
        run = lambda: nm.nm_int_linear(X, T, desc, 0.01, sw, b, Y, status=status)
    for _ in range(3):
        run()
    nm.nm_debug_set_trace(trace)
    run()
    torch.cuda.synchronize()
    nm.nm_debug_set_trace(None)
    rc = nm.nm_poll_status(status)
    tr = trace.cpu().numpy()
    st = tr[:512]
    n = int((st[:, 3] > 0).sum())
    if n == 0:
        print(json.dumps({"error": "no time stamps: this shape runs on a kernel without them (only the CTA-pair kernels have them)"}))
        return 1
    st = st[:n]
    t0 = st[0, 0]
    d = (st[:, :5] - t0).astype(np.float64)
    ok = st[:, 0] > 0     # the last steps of the wide kernel have no load of their own
    med = lambda x: float(np.median(x))
    tl = tr[512:]
    tiles = []
    for i in range(int((tl[:, 0] > 0).sum())):
        row = {"tile": i, "accumulator_full": int(tl[i, 0] - t0), "epilogue_done": int(tl[i, 1] - t0)}
        if tl[i, 2] > 0:
            row.update(second_accumulator_full=int(tl[i, 2] - t0), second_epilogue_done=int(tl[i, 3] - t0))
        elif tl[i, 3:8].sum() > 0:   # the 256-channel pair kernel: the first epilogue warp's phases, summed over the tile
            row["epilogue_warp0_clk"] = dict(zip(["accumulator_chunk_wait", "staging_free_wait", "convert_and_fill", "proxy_fence", "store_issue"],
                                                 (int(x) for x in tl[i, 3:8])))
        tiles.append(row)
    print(json.dumps({"shape": [T, K, OUT], "status": rc, "stages_of_cta0": n,
                      "producer_issue_clk": med((d[:, 1] - d[:, 0])[ok]), "load_issue_to_full_clk": med((d[:, 2] - d[:, 1])[ok]),
                      "gate_to_mma_handoff_clk": med((d[:, 3] - d[:, 2])[ok]), "mma_issue_clk": med(d[:, 4] - d[:, 3]),
                      "clk_per_stage_steady": med(np.diff(d[:, 3])), "first_stage_full_clk": float(d[0, 2]),
                      "last_mma_issued_clk": float(d[-1, 4]), "tiles": tiles,
                      # per stage: when the MMA thread was handed it, and how long its loads took from issue to arrival
                      "stage_handed_to_mma_clk": [int(x) for x in d[:, 3]],
                      "stage_load_clk": [int(x) if k else -1 for x, k in zip(d[:, 2] - d[:, 1], ok)]}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--bits", type=int, default=8, choices=[8, 4], help="weight code width of the 2:4 weights (default 8)")
    ap.add_argument("--out", default="f32", choices=["f32", "int8", "bf16"],
                    help="element type the GEMMs write: fp32 (the headline), int8 with a static scale, bfloat16")
    ap.add_argument("--tokens", type=int, default=TOKENS, help="tokens per GEMM (default: the full workload)")
    ap.add_argument("--skip-cpu", action="store_true", help="leave the CPU-oracle baseline out")
    ap.add_argument("--skip-sweep", action="store_true", help="leave the 24-layer pack sweep out")
    ap.add_argument("--skip-configs", action="store_true", help="leave the timed entries of the other workload configurations out")
    ap.add_argument("--dist-case", type=int, default=0, choices=[0, 4, 8],
                    help="run only a small ADMM-Dist case with this code width (for profiler captures) and exit")
    ap.add_argument("--probe-tma", action="store_true",
                    help="run only the TMA traffic probe of the pair GEMM's tile shapes (no arithmetic) and exit")
    ap.add_argument("--trace-gemm", default="", metavar="TOKENS,K,OUT",
                    help="time stamps of one 2:4 int8 GEMM launch (needs the NM_TRACE build of the library, see trace_gemm)")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="kernel-choice override (nm_debug_set_option) for A/B runs, e.g. no_wide=1 or pack_form=2")
    args = ap.parse_args()
    if args.trace_gemm:
        return trace_gemm(args)
    if args.probe_tma:
        return tma_probe(args)
    if args.dist_case:
        return dist_case(args.dist_case)
    if args.impl == "reference":
        return run_reference(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
