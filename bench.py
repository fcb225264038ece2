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
    """One bounded step of the oracle: pack the attn_out matrix (1024x1024) and run every GEMM of
    the layer on `sample_tokens` tokens.  Returns (seconds, dense-equivalent ops)."""
    import oracle
    import workloads as wl
    n, m, bits = PATTERN
    if "packed" not in state:
        oracle.set_threads(oracle.max_threads())
        rng = np.random.default_rng(2)
        state["packed"], state["X"] = [], []
        for name, k, out in wl.BERT_LARGE_GEMMS:
            W = wl.normal(rng, (out, k), wl.W_STD)
            v, meta, s = oracle.project_pack(W, None, n, m, bits)
            state["packed"].append((oracle.unpack(v, meta, out, k, n, m, bits), s, wl.normal(rng, (out,), wl.W_STD)))
            state["X"].append(wl.random_int8(5, (sample_tokens, k)))
        state["W_pack"], state["U_pack"] = wl.pack_sweep_matrix(3, 1, 1024, 1024)
    t0 = time.perf_counter()
    oracle.project_pack(state["W_pack"], state["U_pack"], n, m, bits)
    ops = 0.0
    for (D, s, b), X in zip(state["packed"], state["X"]):
        oracle.int_linear(X, D, 0.03, s, b, want_acc=False)
        ops += gemm_ops(X.shape[0], D.shape[1], D.shape[0])
    return time.perf_counter() - t0, ops


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
        s, o = oracle_step(sample_tokens, state)
        secs += s
        ops += o
    value = ops / secs / 1e12
    cores = oracle.max_threads()
    sample = f"pack of one 1024x1024 matrix + the four BERT-large GEMMs on the first {sample_tokens} tokens per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def cpu_baseline(budget_s=15.0):
    """The oracle timed on the host cores on a bounded sample (~budget_s of CPU work)."""
    import oracle
    state = {}
    probe, _ = oracle_step(16, state)          # includes building the inputs' first touch
    probe, ops = oracle_step(16, state)
    tokens = int(max(16, min(16384, 16 * budget_s / max(probe, 1e-3))))
    state = {}
    oracle_step(tokens, state)
    secs, ops = oracle_step(tokens, state)
    return {"value": ops / secs / 1e12, "unit": "TOPS", "cores": oracle.max_threads(), "kind": "oracle",
            "sample": f"pack of one 1024x1024 matrix + the four BERT-large GEMMs on the first {tokens} tokens "
                      f"({secs:.1f} s)"}


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

    host = []  # pinned host copies for the end-to-end leg
    devbuf = []
    for name, k, out, W, U, b, Xq in layer:
        hW, hU, hX = (torch.from_numpy(a).pin_memory() for a in (W, U, Xq))
        hY = torch.empty((TOKENS, out), dtype=YDTYPE).pin_memory()
        host.append((hW, hU, hX, hY))
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        d = {"W": hW.to(dev), "U": hU.to(dev), "X": hX.to(dev), "b": torch.from_numpy(b).to(dev),
             "values": torch.empty(vb, dtype=torch.uint8, device=dev),
             "meta": torch.empty(mb // 4, dtype=torch.int32, device=dev),
             "scales": torch.empty(out, dtype=torch.float32, device=dev),
             "Y": torch.empty((TOKENS, out), dtype=YDTYPE, device=dev), "k": k, "out": out, "name": name}
        d["desc"] = nm.make_packed(out, k, n, m, bits, d["values"], d["meta"])
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

    def step(record=False):
        if record:
            e0, e1 = ev(), ev()
            e0.record()
        nm.nm_project_pack_batched(jobs, len(devbuf), ws, ws_bytes, status)
        if record:
            e1.record()
            kernel_events["pack"].append((e0, e1))
        for d in devbuf:
            if record:
                e0, e1 = ev(), ev()
                e0.record()
            if args.out == "f32":
                nm.nm_int_linear(d["X"], TOKENS, d["desc"], sx, d["scales"], d["b"], d["Y"], status=status)
            elif args.out == "int8":
                nm.nm_int_linear_q8(d["X"], TOKENS, d["desc"], sx, d["scales"], d["b"], SY, d["Y"], status=status)
            else:
                nm.nm_int_linear_bf16(d["X"], TOKENS, d["desc"], sx, d["scales"], d["b"], d["Y"], status=status)
            if record:
                e1.record()
                kernel_events[d["name"]].append((e0, e1))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return reduce_max_ms(ms, world, dev)

    # ---- device-resident timing -----------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    t0, t1 = ev(), ev()
    t0.record()
    for k_ in range(args.steps):
        step(record=k_ < 200)
    t1.record()
    barrier()
    ms = max_over_ranks(t0.elapsed_time(t1))
    rc = nm.nm_poll_status(status)
    if rc != nm.NM_OK:
        raise RuntimeError("device status: " + nm.nm_strerror(rc))
    ms_per_step = ms / args.steps
    ops_step = sum(gemm_ops(TOKENS, d["k"], d["out"]) for d in devbuf)
    value = whole_job_tops(ops_step, world, ms_per_step)

    kern = {}
    for name, pairs in kernel_events.items():
        kern[name] = float(np.mean([a.elapsed_time(b) for a, b in pairs])) * 1e3  # microseconds

    # ---- end to end: pinned host buffers in, Y out, every step ------------------------------------
    # Copies run on their own streams: the inputs of step i + 1 go in (after step i's kernels have read the
    # old ones) while the outputs of step i are still leaving; the kernels of step i + 1 wait for both.
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in, ev_comp, ev_out = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()

    def e2e_step():
        s_in.wait_event(ev_comp)
        with torch.cuda.stream(s_in):
            for (hW, hU, hX, hY), d in zip(host, devbuf):
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
            for (hW, hU, hX, hY), d in zip(host, devbuf):
                hY.copy_(d["Y"], non_blocking=True)
            ev_out.record(s_out)

    e2e_steps = max(1, min(args.steps, 5))
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
    h2d = sum(hW.numel() * 4 + hU.numel() * 4 + hX.numel() for hW, hU, hX, hY in host)
    d2h = sum(hY.numel() * YB for hW, hU, hX, hY in host)
    clocks = sampler.stop() if rank == 0 else None

    # ---- projection/pack on the full 24-layer sweep (its own roofline), rank 0 only ---------------
    pack_info = None
    if rank == 0 and not args.skip_sweep:
        pack_info = pack_sweep(nm, torch, dev, status)

    if rank == 0:
        sparse_peak = 4.0 * pk["bf16_tflops"]
        per_kernel = {}
        for d in devbuf:
            us = kern[d["name"]]
            ops, byt = gemm_ops(TOKENS, d["k"], d["out"]), gemm_bytes(TOKENS, d["k"], d["out"], n, m, bits, YB)
            per_kernel[d["name"]] = {
                "us": us, "tops": ops / us / 1e6, "gbs": byt / us / 1e3,
                "frac_sparse_int8_peak_measured": ops / us / 1e6 / sparse_peak,
                "frac_sparse_int8_peak_nominal": ops / us / 1e6 / NOMINAL_SPARSE_INT8_TOPS,
                "frac_hbm_measured": byt / us / 1e3 / pk["hbm_gbs"]}
        pbytes = sum(pack_bytes(d["out"], d["k"], n, m, bits) for d in devbuf)
        per_kernel["pack_layer"] = {"us": kern["pack"], "gbs": pbytes / kern["pack"] / 1e3,
                                    "frac_hbm_measured": pbytes / kern["pack"] / 1e3 / pk["hbm_gbs"]}
        if pack_info:
            per_kernel["pack_sweep"] = pack_info
        # dominant kernel of the step: the FFN1 GEMM launch (longest; bound by the fp32 Y write).
        # `traffic` = dram__bytes_read.sum + dram__bytes_write.sum of one launch at this size (ncu, see
        # profiles/); part of Y is still in the 126 MB L2 when the kernel ends, hence below the algorithmic bytes.
        full_size = TOKENS == 16384 and bits == 8 and args.out == "f32"
        dom = per_kernel["ffn1"]
        # kernel variant the library picks at this size: CTA pairs with resident / streamed weights for
        # int8 2:4; for 4-bit codes the one-CTA kernel whose builder warps widen them in shared memory
        k1 = f"nm_gemm_pair_kernel<sparse,192,{args.out},resident>" if bits == 8 else f"nm_gemm_kernel<sparse,192,{args.out},build-resident>"
        k2 = f"nm_gemm_pair_kernel<sparse,192,{args.out},streamed>" if bits == 8 else f"nm_gemm_kernel<sparse,192,{args.out},build-per-k-block>"
        roofline = {"kernel": k1 + " on ffn1 1024->4096", "bound": "hbm",
                    "achieved": dom["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": dom["gbs"] / pk["hbm_gbs"], "traffic": 241730816 if full_size else None,
                    "algorithmic_bytes": gemm_bytes(TOKENS, 1024, 4096, n, m, bits, YB), "peak_source": pk["source"]}
        f2 = per_kernel["ffn2"]
        roofline_tensor = {"kernel": k2 + " on ffn2 4096->1024", "bound": "tensor",
                           "achieved": f2["tops"], "peak": sparse_peak, "unit": "TOP/s",
                           "frac": f2["tops"] / sparse_peak,
                           "peak_note": "4 x measured bf16 burst (nominal int8-sparse : bf16-dense ratio)",
                           "frac_of_nominal_9000": f2["tops"] / NOMINAL_SPARSE_INT8_TOPS,
                           "traffic": 113428480 if full_size else None}
        line = {"metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
                "config": {"workload": WORKLOAD if TOKENS == 16384 else WORKLOAD + f" (reduced to {TOKENS} tokens)", "tokens": TOKENS, "pattern": "2:4", "bits": bits, "out": args.out,
                           "l2": "inputs+outputs per step (715 MB) exceed L2; no flush needed"},
                "clocks": clocks,
                "e2e": {"value": whole_job_tops(ops_step, world, e2e_ms), "unit": "TOPS",
                        "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
                "gpu_launches": 5 * args.steps,
                "roofline": roofline, "roofline_tensor": roofline_tensor, "kernels": per_kernel}
        if pack_info:
            line["roofline_pack"] = {"kernel": "pack_kernel<2,4,8> on the 24-layer sweep", "bound": "hbm",
                                     "achieved": pack_info["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                                     "frac": pack_info["gbs"] / pk["hbm_gbs"],
                                     "frac_of_nominal_8000": pack_info["gbs"] / NOMINAL_HBM_GBS, "traffic": 2549617536,
                                     "algorithmic_bytes": pack_info["bytes"]}
            adm = pack_info["admm_step_2:4/8b"]
            line["roofline_admm"] = {"kernel": "pack_kernel<2,4,8,dense outputs> (ADMM step: Z and U_next) on the 24-layer sweep",
                                     "bound": "hbm", "achieved": adm["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                                     "frac": adm["gbs"] / pk["hbm_gbs"], "traffic": 4771902805,
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
    clocks = torch.zeros((148, 4), dtype=torch.int64, device=dev)

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
    # everything resident in L2: a small problem walked five times
    case("L2-resident 256x192", OUT, K, 19 * 192, 128, 128, 96, 2, 5, repeat=5, stores=0, producers=2)
    case("L2-resident 512x224", OUT, K, 37 * 224, 256, 64, 112, 1, 6, repeat=5, stores=0, producers=2)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--bits", type=int, default=8, choices=[8, 4], help="weight code width of the 2:4 weights (default 8)")
    ap.add_argument("--out", default="f32", choices=["f32", "int8", "bf16"],
                    help="element type the GEMMs write: fp32 (the headline), int8 with a static scale, bfloat16")
    ap.add_argument("--tokens", type=int, default=TOKENS, help="tokens per GEMM (default: the full workload)")
    ap.add_argument("--skip-cpu", action="store_true", help="leave the CPU-oracle baseline out")
    ap.add_argument("--skip-sweep", action="store_true", help="leave the 24-layer pack sweep out")
    ap.add_argument("--dist-case", type=int, default=0, choices=[0, 4, 8],
                    help="run only a small ADMM-Dist case with this code width (for profiler captures) and exit")
    ap.add_argument("--probe-tma", action="store_true",
                    help="run only the TMA traffic probe of the pair GEMM's tile shapes (no arithmetic) and exit")
    args = ap.parse_args()
    if args.probe_tma:
        return tma_probe(args)
    if args.dist_case:
        return dist_case(args.dist_case)
    if args.impl == "reference":
        return run_reference(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
