"""The scratch-free batched projection gives the same bytes as the one that takes a workspace.

Meant for hosts that must not allocate device memory while running (pooled-memory servers,
real-time loops, plug-ins called from another framework's stream).  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import workloads as wl

pytestmark = pytest.mark.gpu


def _jobs(nm, dev, seed, n, m, bits):
    # more than eight matrices share one kernel variant, so the job table really lives in device memory (smaller
    # batches pass it in the kernel's parameters and would leave the library's fixed array unused)
    shapes = [(96, 1024), (40, 4096), (8, 8192), (50, 768)] * 3
    jobs = []
    for i, (out, k) in enumerate(shapes):
        W, U = wl.pack_sweep_matrix(seed, i, out, k)
        vb, mb = nm.nm_packed_sizes(out, k, n, m, bits)
        jobs.append((torch.from_numpy(W).to(dev), torch.from_numpy(U).to(dev), n, m, bits,
                     torch.zeros(vb, dtype=torch.uint8, device=dev),
                     torch.zeros(max(mb // 4, 1), dtype=torch.int32, device=dev),
                     torch.zeros(out, dtype=torch.float32, device=dev)))
    return jobs


def test_noalloc_matches_workspace_variant_twice_in_a_row():
    import paper_2206_15014_b200 as nm
    dev = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # two consecutive calls with different jobs: the second must not see the first one's table
    for call, (seed, n, m, bits) in enumerate([(11, 2, 4, 8), (12, 1, 4, 4)]):
        ref_jobs = _jobs(nm, dev, seed, n, m, bits)
        ws_bytes = nm.nm_pack_workspace_bytes(len(ref_jobs))
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        nm.nm_project_pack_batched(nm.make_pack_jobs(ref_jobs), len(ref_jobs), ws, ws_bytes, status)
        new_jobs = _jobs(nm, dev, seed, n, m, bits)
        nm.nm_project_pack_batched_noalloc(nm.make_pack_jobs(new_jobs), len(new_jobs), status)
        assert nm.nm_poll_status(status) == nm.NM_OK
        for a, b in zip(ref_jobs, new_jobs):
            for x, y in zip(a[5:], b[5:]):  # values, metadata, scales: bit for bit
                assert torch.equal(x, y), f"call {call}: outputs differ"
            assert a[5].any() and a[7].abs().sum() > 0


def test_noalloc_rejects_too_many_jobs():
    import paper_2206_15014_b200 as nm
    dev = torch.device("cuda:0")
    jobs = _jobs(nm, dev, 13, 2, 4, 8)[:1] * (nm.NM_NOALLOC_MAX_JOBS + 1)
    with pytest.raises(nm.NmError) as e:
        nm.nm_project_pack_batched_noalloc(nm.make_pack_jobs(jobs), len(jobs))
    assert e.value.code == nm.NM_ERR_UNSUPPORTED
    nm.nm_project_pack_batched_noalloc(nm.make_pack_jobs(jobs[:1]), 0)  # nothing to do
