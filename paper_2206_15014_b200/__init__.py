"""Python binding of libnmsparse.so: argument marshalling only.

Every function has the name and the argument order of its C entry point (include/nmsparse.h) and
takes torch CUDA tensors (used purely as device buffers) or plain integers.  All arithmetic runs in
the library's CUDA kernels.  There is no CPU fallback: importing this package fails when the
library has not been built (run ``python paper_2206_15014_b200/build.py``).
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# NMSPARSE_LIB selects another build of the same library (the -DNM_TRACE build with time stamps in its kernels, the
# build with short device-side wait limits that the timeout test uses); the default is the product library.
LIB_PATH = os.environ.get("NMSPARSE_LIB") or os.path.join(_HERE, "libnmsparse.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_2206_15014_b200/build.py` "
        "(there is no fallback path)")

_lib = ctypes.CDLL(LIB_PATH)

NM_OK = 0
NM_ERR_NULL, NM_ERR_SHAPE, NM_ERR_UNSUPPORTED, NM_ERR_ALIGN = -1, -2, -3, -4
NM_ERR_WORKSPACE, NM_ERR_CUDA, NM_ERR_NONFINITE, NM_ERR_TIMEOUT = -5, -6, -7, -8

EXPORTS = (
    "nm_packed_sizes", "nm_project_pack", "nm_project_pack_batched", "nm_pack_workspace_bytes",
    "nm_project_pack_batched_noalloc", "nm_admm_project", "nm_admm_project_batched", "nm_admm_workspace_bytes",
    "nm_project_pack_grouped", "nm_admm_project_grouped", "nm_project_pack_grouped_batched",
    "nm_admm_project_grouped_batched",
    "nm_dist_scales", "nm_project_pack_dist", "nm_admm_project_dist", "nm_project_pack_dist_batched", "nm_admm_project_dist_batched",
    "nm_int_linear", "nm_int_linear_dsx", "nm_int_linear_acc", "nm_int_linear_q8", "nm_int_linear_bf16",
    "nm_int_linear_workspace_bytes",
    "nm_int_linear_check", "nm_absmax", "nm_quantize_act", "nm_poll_status", "nm_strerror",
    "nm_last_cuda_error", "nm_version", "nm_bits_per_param", "nm_encoder_cost", "nm_pair_tile_plan",
    "nm_probe_tma_stream", "nm_debug_set_trace", "nm_debug_set_option",
)


class nm_packed_t(ctypes.Structure):
    _fields_ = [("out", ctypes.c_int32), ("in_", ctypes.c_int32), ("n", ctypes.c_int32),
                ("m", ctypes.c_int32), ("bits", ctypes.c_int32), ("values", ctypes.c_void_p),
                ("meta", ctypes.c_void_p)]


class nm_pack_job_t(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("U", ctypes.c_void_p), ("out", ctypes.c_int32),
                ("in_", ctypes.c_int32), ("n", ctypes.c_int32), ("m", ctypes.c_int32),
                ("bits", ctypes.c_int32), ("values", ctypes.c_void_p), ("meta", ctypes.c_void_p),
                ("scales", ctypes.c_void_p)]


class nm_admm_job_t(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("U", ctypes.c_void_p), ("out", ctypes.c_int32),
                ("in_", ctypes.c_int32), ("n", ctypes.c_int32), ("m", ctypes.c_int32),
                ("bits", ctypes.c_int32), ("Z", ctypes.c_void_p), ("U_next", ctypes.c_void_p),
                ("values", ctypes.c_void_p), ("meta", ctypes.c_void_p), ("scales", ctypes.c_void_p)]


_vp, _i, _sz, _f = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_float
_lib.nm_packed_sizes.argtypes = [_i] * 5 + [ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
_lib.nm_project_pack.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp]
_lib.nm_project_pack_batched.argtypes = [ctypes.POINTER(nm_pack_job_t), _i, _vp, _sz, _vp, _vp]
_lib.nm_project_pack_batched_noalloc.argtypes = [ctypes.POINTER(nm_pack_job_t), _i, _vp, _vp]
_lib.nm_admm_project_grouped_batched.argtypes = [ctypes.POINTER(nm_admm_job_t), _i, _i, _vp, _sz, _vp, _vp]
_lib.nm_project_pack_grouped_batched.argtypes = [ctypes.POINTER(nm_pack_job_t), _i, _i, _vp, _sz, _vp, _vp]
_lib.nm_project_pack_grouped.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp]
_lib.nm_admm_project_grouped.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nm_dist_scales.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp]
_lib.nm_project_pack_dist.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp]
_lib.nm_admm_project_dist.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nm_project_pack_dist_batched.argtypes = [ctypes.POINTER(nm_pack_job_t), _i, _i, _vp, _sz, _vp, _vp]
_lib.nm_admm_project_dist_batched.argtypes = [ctypes.POINTER(nm_admm_job_t), _i, _i, _vp, _sz, _vp, _vp]
_lib.nm_admm_project_batched.argtypes = [ctypes.POINTER(nm_admm_job_t), _i, _vp, _sz, _vp, _vp]
_lib.nm_admm_project.argtypes = [_vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nm_admm_workspace_bytes.argtypes = [_i]
_lib.nm_admm_workspace_bytes.restype = _sz
_lib.nm_pack_workspace_bytes.argtypes = [_i]
_lib.nm_pack_workspace_bytes.restype = _sz
_lib.nm_int_linear.argtypes = [_vp, _i, ctypes.POINTER(nm_packed_t), _f, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.nm_int_linear_dsx.argtypes = [_vp, _i, ctypes.POINTER(nm_packed_t), _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.nm_int_linear_acc.argtypes = [_vp, _i, ctypes.POINTER(nm_packed_t), _vp, _vp, _sz, _vp, _vp]
_lib.nm_int_linear_q8.argtypes = [_vp, _i, ctypes.POINTER(nm_packed_t), _f, _vp, _vp, _f, _vp, _vp, _sz, _vp, _vp]
_lib.nm_int_linear_bf16.argtypes = [_vp, _i, ctypes.POINTER(nm_packed_t), _f, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.nm_int_linear_workspace_bytes.argtypes = [_i] * 6
_lib.nm_int_linear_workspace_bytes.restype = _sz
_lib.nm_int_linear_check.argtypes = [_i] * 6
_lib.nm_probe_tma_stream.argtypes = [_vp, _i, _i, _vp, _i, _i, _vp] + [_i] * 12 + [_vp, _vp, _vp, _vp]
_lib.nm_debug_set_trace.argtypes = [_vp]
_lib.nm_debug_set_option.argtypes = [ctypes.c_char_p, _i]
_lib.nm_absmax.argtypes = [_vp, _sz, _vp, _vp]
_lib.nm_quantize_act.argtypes = [_vp, _sz, _vp, _vp, _vp, _vp]
_lib.nm_poll_status.argtypes = [_vp, _vp]
_lib.nm_bits_per_param.argtypes = [_i] * 4
_lib.nm_bits_per_param.restype = ctypes.c_double
_lib.nm_strerror.argtypes = [_i]
_lib.nm_strerror.restype = ctypes.c_char_p
_lib.nm_last_cuda_error.restype = ctypes.c_char_p


class NmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        extra = nm_last_cuda_error() if code == NM_ERR_CUDA else ""
        super().__init__(f"{where}: {nm_strerror(code)} ({code}) {extra}".strip())


def _chk(code, where):
    if code != NM_OK:
        raise NmError(code, where)


def _ptr(t):
    # a plain int converts to void* through the declared argtypes; no ctypes object per argument
    return None if t is None else t.data_ptr()


def _stream(stream=None):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(stream)


def nm_strerror(code):
    return _lib.nm_strerror(int(code)).decode()


def nm_last_cuda_error():
    return _lib.nm_last_cuda_error().decode()


def nm_version():
    return int(_lib.nm_version())


def nm_packed_sizes(out, in_, n, m, bits):
    vb, mb = _sz(), _sz()
    _chk(_lib.nm_packed_sizes(out, in_, n, m, bits, ctypes.byref(vb), ctypes.byref(mb)), "nm_packed_sizes")
    return vb.value, mb.value


def nm_project_pack(W, U, out, in_, n, m, bits, values, meta, scales, status=None, stream=None):
    _chk(_lib.nm_project_pack(_ptr(W), _ptr(U), out, in_, n, m, bits, _ptr(values), _ptr(meta),
                              _ptr(scales), _ptr(status), _stream(stream)), "nm_project_pack")


def nm_pack_workspace_bytes(njobs):
    return int(_lib.nm_pack_workspace_bytes(njobs))


def make_pack_jobs(jobs):
    """jobs: iterable of (W, U|None, n, m, bits, values, meta|None, scales) -> ctypes job array."""
    jobs = list(jobs)
    arr = (nm_pack_job_t * len(jobs))()
    for a, (W, U, n, m, bits, values, meta, scales) in zip(arr, jobs):
        a.W, a.U = W.data_ptr(), (U.data_ptr() if U is not None else None)
        a.out, a.in_, a.n, a.m, a.bits = W.shape[0], W.shape[1], n, m, bits
        a.values, a.meta, a.scales = values.data_ptr(), (meta.data_ptr() if meta is not None else None), scales.data_ptr()
    return arr


def nm_project_pack_batched(job_array, njobs, ws, ws_bytes, status=None, stream=None):
    _chk(_lib.nm_project_pack_batched(job_array, njobs, _ptr(ws), ws_bytes, _ptr(status), _stream(stream)),
         "nm_project_pack_batched")


NM_NOALLOC_MAX_JOBS = 1024


def nm_project_pack_batched_noalloc(job_array, njobs, status=None, stream=None):
    """Batched projection whose job table sits in a fixed array inside the library (at most
    NM_NOALLOC_MAX_JOBS jobs): for callers that may not allocate device memory.  Calls that overlap
    on the GPU share that table and must be serialised by the caller."""
    _chk(_lib.nm_project_pack_batched_noalloc(job_array, njobs, _ptr(status), _stream(stream)),
         "nm_project_pack_batched_noalloc")


def make_packed(out, in_, n, m, bits, values, meta):
    return nm_packed_t(out, in_, n, m, bits, values.data_ptr(), meta.data_ptr() if meta is not None else None)


def nm_admm_project(W, U, out, in_, n, m, bits, Z, U_next=None, values=None, meta=None, scales=None,
                    status=None, stream=None):
    _chk(_lib.nm_admm_project(_ptr(W), _ptr(U), out, in_, n, m, bits, _ptr(Z), _ptr(U_next), _ptr(values),
                              _ptr(meta), _ptr(scales), _ptr(status), _stream(stream)), "nm_admm_project")


NM_DIST_MAX_CANDIDATES = 32


def nm_dist_scales(W, U, out, in_, n, m, bits, ncand, scales, cand=None, status=None, stream=None):
    _chk(_lib.nm_dist_scales(_ptr(W), _ptr(U), out, in_, n, m, bits, ncand, _ptr(scales), _ptr(cand), _ptr(status),
                             _stream(stream)), "nm_dist_scales")


def nm_project_pack_dist(W, U, out, in_, n, m, bits, ncand, values, meta, scales, status=None, stream=None):
    _chk(_lib.nm_project_pack_dist(_ptr(W), _ptr(U), out, in_, n, m, bits, ncand, _ptr(values), _ptr(meta),
                                   _ptr(scales), _ptr(status), _stream(stream)), "nm_project_pack_dist")


def nm_admm_project_dist(W, U, out, in_, n, m, bits, ncand, Z, U_next, values, meta, scales, status=None,
                         stream=None):
    _chk(_lib.nm_admm_project_dist(_ptr(W), _ptr(U), out, in_, n, m, bits, ncand, _ptr(Z), _ptr(U_next), _ptr(values),
                                   _ptr(meta), _ptr(scales), _ptr(status), _stream(stream)), "nm_admm_project_dist")


def nm_project_pack_dist_batched(jobs, njobs, ncand, ws, ws_bytes, status=None, stream=None):
    _chk(_lib.nm_project_pack_dist_batched(jobs, njobs, ncand, _ptr(ws), ws_bytes, _ptr(status), _stream(stream)),
         "nm_project_pack_dist_batched")


def nm_admm_project_dist_batched(jobs, njobs, ncand, ws, ws_bytes, status=None, stream=None):
    _chk(_lib.nm_admm_project_dist_batched(jobs, njobs, ncand, _ptr(ws), ws_bytes, _ptr(status), _stream(stream)),
         "nm_admm_project_dist_batched")


def nm_project_pack_grouped(W, U, out, in_, n, m, bits, group_rows, values, meta, scales, status=None, stream=None):
    _chk(_lib.nm_project_pack_grouped(_ptr(W), _ptr(U), out, in_, n, m, bits, group_rows, _ptr(values), _ptr(meta),
                                      _ptr(scales), _ptr(status), _stream(stream)), "nm_project_pack_grouped")


def nm_project_pack_grouped_batched(jobs, njobs, group_rows, ws, ws_bytes, status=None, stream=None):
    _chk(_lib.nm_project_pack_grouped_batched(jobs, njobs, group_rows, _ptr(ws), ws_bytes, _ptr(status),
                                              _stream(stream)), "nm_project_pack_grouped_batched")


def nm_admm_project_grouped_batched(jobs, njobs, group_rows, ws, ws_bytes, status=None, stream=None):
    _chk(_lib.nm_admm_project_grouped_batched(jobs, njobs, group_rows, _ptr(ws), ws_bytes, _ptr(status),
                                              _stream(stream)), "nm_admm_project_grouped_batched")


def nm_admm_project_grouped(W, U, out, in_, n, m, bits, group_rows, Z, U_next, values, meta, scales,
                            status=None, stream=None):
    _chk(_lib.nm_admm_project_grouped(_ptr(W), _ptr(U), out, in_, n, m, bits, group_rows, _ptr(Z), _ptr(U_next),
                                      _ptr(values), _ptr(meta), _ptr(scales), _ptr(status), _stream(stream)),
         "nm_admm_project_grouped")


def nm_admm_workspace_bytes(njobs):
    return int(_lib.nm_admm_workspace_bytes(njobs))


def make_admm_jobs(jobs):
    """jobs: iterable of (W, U, n, m, bits, Z, U_next, values, meta, scales) tensors / None -> ctypes array."""
    dp = lambda t: None if t is None else t.data_ptr()
    arr = (nm_admm_job_t * len(jobs))()
    for i, (W, U, n, m, bits, Z, Un, v, mt, sc) in enumerate(jobs):
        arr[i] = nm_admm_job_t(dp(W), dp(U), W.shape[0], W.shape[1], n, m, bits, dp(Z), dp(Un), dp(v), dp(mt), dp(sc))
    return arr


def nm_admm_project_batched(jobs, njobs, ws, ws_bytes, status=None, stream=None):
    _chk(_lib.nm_admm_project_batched(jobs, njobs, _ptr(ws), ws_bytes, _ptr(status), _stream(stream)),
         "nm_admm_project_batched")


def nm_int_linear_workspace_bytes(tokens, out, in_, n, m, bits):
    return int(_lib.nm_int_linear_workspace_bytes(tokens, out, in_, n, m, bits))


def nm_int_linear_check(tokens, out, in_, n, m, bits):
    return int(_lib.nm_int_linear_check(tokens, out, in_, n, m, bits))


def nm_int_linear(X, tokens, W, sx, sw, bias, Y, ws=None, ws_bytes=0, status=None, stream=None):
    _chk(_lib.nm_int_linear(_ptr(X), tokens, ctypes.byref(W), float(sx), _ptr(sw), _ptr(bias), _ptr(Y),
                            _ptr(ws), ws_bytes, _ptr(status), _stream(stream)), "nm_int_linear")


def nm_int_linear_dsx(X, tokens, W, sx_dev, sw, bias, Y, absmax_out=None, ws=None, ws_bytes=0,
                      status=None, stream=None):
    _chk(_lib.nm_int_linear_dsx(_ptr(X), tokens, ctypes.byref(W), _ptr(sx_dev), _ptr(sw), _ptr(bias),
                                _ptr(Y), _ptr(absmax_out), _ptr(ws), ws_bytes, _ptr(status),
                                _stream(stream)), "nm_int_linear_dsx")


def nm_int_linear_acc(X, tokens, W, ACC, ws=None, ws_bytes=0, status=None, stream=None):
    _chk(_lib.nm_int_linear_acc(_ptr(X), tokens, ctypes.byref(W), _ptr(ACC), _ptr(ws), ws_bytes,
                                _ptr(status), _stream(stream)), "nm_int_linear_acc")


def nm_int_linear_q8(X, tokens, W, sx, sw, bias, sy, Yq, ws=None, ws_bytes=0, status=None, stream=None):
    _chk(_lib.nm_int_linear_q8(_ptr(X), tokens, ctypes.byref(W), float(sx), _ptr(sw), _ptr(bias), float(sy),
                               _ptr(Yq), _ptr(ws), ws_bytes, _ptr(status), _stream(stream)), "nm_int_linear_q8")


def nm_int_linear_bf16(X, tokens, W, sx, sw, bias, Ybf16, ws=None, ws_bytes=0, status=None, stream=None):
    _chk(_lib.nm_int_linear_bf16(_ptr(X), tokens, ctypes.byref(W), float(sx), _ptr(sw), _ptr(bias),
                                 _ptr(Ybf16), _ptr(ws), ws_bytes, _ptr(status), _stream(stream)),
         "nm_int_linear_bf16")


class nm_component_cfg_t(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("m", ctypes.c_int32), ("bits", ctypes.c_int32)]


def nm_pair_tile_plan(n_tok_tiles, n_out_tiles, pairs, resident, band_request=0):
    """-> (band, start list [pairs + 1], tile_out list, tile_tok list): the pair kernel's tile walk (host only)."""
    n = n_tok_tiles * n_out_tiles
    start = (ctypes.c_int * (pairs + 1))()
    to, tt = (ctypes.c_int * max(n, 1))(), (ctypes.c_int * max(n, 1))()
    band = _lib.nm_pair_tile_plan(n_tok_tiles, n_out_tiles, pairs, int(bool(resident)), band_request, start, to, tt)
    _chk(min(band, 0), "nm_pair_tile_plan")
    return band, list(start), list(to)[:n], list(tt)[:n]


def nm_bits_per_param(n, m, bits, index_bits=-1):
    return float(_lib.nm_bits_per_param(n, m, bits, index_bits))


def nm_encoder_cost(cfg, index_bits=-1):
    """cfg: six (n, m, bits) for Q, K, V, attention output, FFN1, FFN2 -> (compression, mac_reduction)."""
    arr = (nm_component_cfg_t * 6)(*[nm_component_cfg_t(*c) for c in cfg])
    comp, red = ctypes.c_double(), ctypes.c_double()
    _chk(_lib.nm_encoder_cost(arr, index_bits, ctypes.byref(comp), ctypes.byref(red)), "nm_encoder_cost")
    return comp.value, red.value


def nm_probe_tma_stream(W, w_rows, w_row_bytes, X, tokens, k_bytes, Y, a_rows, a_row_bytes, b_rows, b_slices, stages,
                        band=0, repeat=1, delay_clocks=0, loads=3, stores=1, producers=1, poll=0, clocks=None, trace=None,
                        status=None, stream=None):
    """Replays the pair GEMM's tile walk with its TMA boxes and no arithmetic; returns the number of CTAs launched
    (`clocks`, int64 [CTAs, 4], receives clock64 at start / end and the global timer at start / end of every CTA)."""
    rc = _lib.nm_probe_tma_stream(_ptr(W), w_rows, w_row_bytes, _ptr(X), tokens, k_bytes, _ptr(Y), a_rows, a_row_bytes,
                                  b_rows, b_slices, stages, band, repeat, delay_clocks, loads, stores, producers, poll, _ptr(clocks), _ptr(trace),
                                  _ptr(status), _stream(stream))
    if rc < 0:
        raise NmError(rc, "nm_probe_tma_stream")
    return int(rc)


def nm_debug_set_option(name, value):
    """Kernel-choice override for measurements and tests (see nmsparse.h); 0 restores the library's own choice."""
    _chk(_lib.nm_debug_set_option(name.encode(), int(value)), "nm_debug_set_option")


def nm_debug_set_trace(buffer):
    """Hands a zeroed int64 [576, 8] device tensor (or None) to the GEMM launches of an NM_TRACE build."""
    _chk(_lib.nm_debug_set_trace(_ptr(buffer)), "nm_debug_set_trace")


def nm_absmax(Y, count, absmax, stream=None):
    _chk(_lib.nm_absmax(_ptr(Y), count, _ptr(absmax), _stream(stream)), "nm_absmax")


def nm_quantize_act(Y, count, absmax, Xq, sx_out=None, stream=None):
    _chk(_lib.nm_quantize_act(_ptr(Y), count, _ptr(absmax), _ptr(Xq), _ptr(sx_out), _stream(stream)),
         "nm_quantize_act")


def nm_poll_status(status=None, stream=None):
    """Synchronises the stream and returns the NM_* code held in the device status word."""
    return int(_lib.nm_poll_status(_ptr(status), _stream(stream)))
