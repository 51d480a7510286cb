"""Thin ctypes binding over libkata.so (argument marshalling only; every step runs in the CUDA
library).  Function names mirror the C ABI of include/kata.h.

Tensors are torch CUDA tensors (or pinned host tensors for ``kata_fwd_host``); torch is used for
device memory and streams only.  There is no CPU fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libkata.so")

KATA_F32, KATA_BF16 = 0, 1
KATA_LAYOUT_DIRECT, KATA_LAYOUT_PACKED = 0, 1
KATA_SEQUENTIAL, KATA_SCAN, KATA_INTER_AUTO = 0, 1, 2
KATA_IMPL_AUTO, KATA_IMPL_SIMT, KATA_IMPL_TENSOR = 0, 1, 2
KATA_FN_QUADRATIC, KATA_FN_CHUNKED, KATA_FN_CHUNK_STATE_SCAN, KATA_FN_DECODE_STEP = 0, 1, 2, 3
KATA_FN_BWD_QUADRATIC = 4
KATA_FN_BWD_CHUNKED = 5
KATA_FN_HOST_IO = 0x100
KATA_OK, KATA_ERR_INVALID_ARG, KATA_ERR_UNSUPPORTED_SHAPE, KATA_ERR_WORKSPACE_TOO_SMALL, KATA_ERR_DEVICE_TIMEOUT = 0, -1, -2, -4, -7

EXPORTS = ("kata_fwd_quadratic", "kata_fwd_chunked", "kata_chunk_state_scan", "kata_chunk_state_scan_static",
           "kata_fwd_host", "kata_decode_step", "kata_bwd_quadratic", "kata_bwd_chunked",
           "kata_workspace_bytes", "kata_scan_plan", "kata_host_plan", "kata_last_launch_count", "kata_last_impl",
           "kata_status_string",
           "kata_version")


class KataOpts(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("dtype", ctypes.c_int32),
        ("feature_order", ctypes.c_int32),
        ("state_layout", ctypes.c_int32),
        ("inter_chunk", ctypes.c_int32),
        ("impl", ctypes.c_int32),
        ("scan_group", ctypes.c_int32),
        ("feature_groups", ctypes.c_int32),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
        ("s_pre", ctypes.c_void_p),
        ("z_pre", ctypes.c_void_p),
        ("device_status", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
        ("s_init", ctypes.c_void_p),
        ("z_init", ctypes.c_void_p),
    ]


class KataError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libkata.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2607_17419_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    ptr, i = ctypes.c_void_p, ctypes.c_int
    fwd_args = [ptr, ptr, ptr, ptr, i, i, i, i, i, i, ctypes.POINTER(KataOpts)]
    for name in ("kata_fwd_quadratic", "kata_fwd_chunked", "kata_chunk_state_scan", "kata_chunk_state_scan_static"):
        getattr(L, name).argtypes = fwd_args
        getattr(L, name).restype = i
    L.kata_fwd_host.argtypes = [i] + fwd_args
    L.kata_fwd_host.restype = i
    L.kata_decode_step.argtypes = [ptr, ptr, ptr, ptr, ptr, ptr, i, i, i, i, ctypes.POINTER(KataOpts)]
    L.kata_decode_step.restype = i
    L.kata_bwd_quadratic.argtypes = [ptr] * 7 + [i] * 5 + [ctypes.POINTER(KataOpts)]
    L.kata_bwd_quadratic.restype = i
    L.kata_bwd_chunked.argtypes = [ptr] * 7 + [i] * 6 + [ctypes.POINTER(KataOpts)]
    L.kata_bwd_chunked.restype = i
    L.kata_workspace_bytes.argtypes = [i, i, i, i, i, i, i, ctypes.POINTER(KataOpts)]
    L.kata_workspace_bytes.restype = ctypes.c_size_t
    L.kata_scan_plan.argtypes = [i, i, i, i, i, i, i, ctypes.POINTER(KataOpts)] + [ctypes.POINTER(i)] * 3
    L.kata_scan_plan.restype = i
    L.kata_host_plan.argtypes = [i, i, i, i, i, i, i, ctypes.POINTER(KataOpts)] + [ctypes.POINTER(i)] * 2
    L.kata_host_plan.restype = i
    L.kata_last_launch_count.argtypes = []
    L.kata_last_launch_count.restype = i
    L.kata_last_impl.argtypes = []
    L.kata_last_impl.restype = i
    L.kata_status_string.argtypes = [i]
    L.kata_status_string.restype = ctypes.c_char_p
    L.kata_version.argtypes = []
    L.kata_version.restype = i
    L.kata_selftest_wait_timeout.argtypes = [ptr, ptr, ctypes.c_uint, ptr]
    L.kata_selftest_wait_timeout.restype = i
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().kata_status_string(status).decode()


def make_opts(dtype: int, *, feature_order: int = 2, state_layout: int = KATA_LAYOUT_DIRECT,
              inter_chunk: int = KATA_SEQUENTIAL, impl: int = KATA_IMPL_AUTO, scan_group: int = 0,
              feature_groups: int = 0,
              workspace: int = 0, workspace_bytes: int = 0, s_pre: int = 0, z_pre: int = 0,
              device_status: int = 0, stream: int = 0, s_init: int = 0, z_init: int = 0) -> KataOpts:
    o = KataOpts()
    o.struct_size = ctypes.sizeof(KataOpts)
    o.dtype, o.feature_order, o.state_layout = dtype, feature_order, state_layout
    o.inter_chunk, o.impl, o.scan_group = inter_chunk, impl, scan_group
    o.feature_groups = feature_groups
    o.workspace, o.workspace_bytes = workspace or None, workspace_bytes
    o.s_pre, o.z_pre = s_pre or None, z_pre or None
    o.device_status, o.stream = device_status or None, stream or None
    o.s_init, o.z_init = s_init or None, z_init or None
    return o


def kata_workspace_bytes(fn: int, B, H, T, d_k, d_v, C, opts: KataOpts) -> int:
    return int(lib().kata_workspace_bytes(fn, B, H, T, d_k, d_v, C, ctypes.byref(opts)))


def kata_scan_plan(fn: int, B, H, T, d_k, d_v, C, opts: KataOpts):
    """(n_groups, chunks_per_group, scan_rounds) the library would use."""
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    st = lib().kata_scan_plan(fn, B, H, T, d_k, d_v, C, ctypes.byref(opts), ctypes.byref(a), ctypes.byref(b),
                              ctypes.byref(c))
    if st != 0:
        raise KataError(st, "kata_scan_plan")
    return a.value, b.value, c.value


def kata_host_plan(fn: int, B, H, T, d_k, d_v, C, opts: KataOpts):
    """(pieces, tokens per piece) the host-buffer entry would work in."""
    a, b = ctypes.c_int(), ctypes.c_int()
    st = lib().kata_host_plan(fn, B, H, T, d_k, d_v, C, ctypes.byref(opts), ctypes.byref(a), ctypes.byref(b))
    if st != 0:
        raise KataError(st, "kata_host_plan")
    return a.value, b.value


def kata_selftest_wait_timeout(device_status, report, max_polls: int = 1000, stream=None) -> int:
    """Test hook (csrc/kata_selftest.h): one warp runs both bounded waits on a barrier nobody arrives at.

    `device_status` is an int32 CUDA tensor of one element (or None), `report` one of eight (the last is the flag in
    global memory that the flag wait is tried on: 0 on entry).  Returns the status code.
    """
    import torch
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    return int(lib().kata_selftest_wait_timeout(device_status.data_ptr() if device_status is not None else None,
                                                report.data_ptr() if report is not None else None, max_polls, stream))


def kata_last_launch_count() -> int:
    return int(lib().kata_last_launch_count())


def kata_last_impl() -> int:
    return int(lib().kata_last_impl())


def kata_version() -> int:
    return int(lib().kata_version())


# ---------------------------------------------------------------------------
# tensor-level wrappers
# ---------------------------------------------------------------------------

_FN_NAMES = {KATA_FN_QUADRATIC: "kata_fwd_quadratic", KATA_FN_CHUNKED: "kata_fwd_chunked",
             KATA_FN_CHUNK_STATE_SCAN: "kata_chunk_state_scan"}


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return KATA_F32
    if t.dtype == torch.bfloat16:
        return KATA_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


class Workspace:
    """A reusable device scratch buffer (torch allocation, grown on demand)."""

    def __init__(self):
        self.buf = None

    def get(self, nbytes: int, device):
        import torch
        if nbytes == 0:
            return 0, 0
        if self.buf is None or self.buf.numel() < nbytes or self.buf.device != device:
            self.buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        return self.buf.data_ptr(), self.buf.numel()


_default_ws = Workspace()


def _call(fn: int, q, k, v, out, C: int, *, host_io: bool = False, workspace: Optional[Workspace] = None,
          s_pre=None, z_pre=None, s_init=None, z_init=None, device_status=None, stream=None, **opt_kw):
    import torch
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
        raise ValueError("q, k, v must be contiguous [B,H,T,d]")
    B, H, T, d_k = q.shape
    d_v = v.shape[-1]
    if out is None:
        out = torch.empty_like(v)
    dev = torch.device("cuda", torch.cuda.current_device()) if host_io else q.device
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    opts = make_opts(_dtype_code(q), stream=stream,
                     s_pre=s_pre.data_ptr() if s_pre is not None else 0,
                     z_pre=z_pre.data_ptr() if z_pre is not None else 0,
                     s_init=s_init.data_ptr() if s_init is not None else 0,
                     z_init=z_init.data_ptr() if z_init is not None else 0,
                     device_status=device_status.data_ptr() if device_status is not None else 0, **opt_kw)
    need = kata_workspace_bytes(fn | (KATA_FN_HOST_IO if host_io else 0), B, H, T, d_k, d_v, C, opts)
    ws = workspace if workspace is not None else _default_ws
    ptr, size = ws.get(need, dev)
    opts.workspace, opts.workspace_bytes = ptr or None, size
    args = (q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), B, H, T, d_k, d_v, C, ctypes.byref(opts))
    if host_io:
        st = lib().kata_fwd_host(fn, *args)
        name = "kata_fwd_host"
    else:
        name = _FN_NAMES[fn]
        st = getattr(lib(), name)(*args)
    if st != 0:
        raise KataError(st, name)
    return out


def kata_fwd_quadratic(q, k, v, out=None, C: int = 64, **kw):
    """Quadratic forward; q,k [B,H,T,d_k], v [B,H,T,d_v] CUDA tensors (fp32 or bf16)."""
    return _call(KATA_FN_QUADRATIC, q, k, v, out, C, **kw)


def kata_fwd_chunked(q, k, v, out=None, C: int = 64, **kw):
    """Chunked-state forward; inter_chunk=KATA_SEQUENTIAL (default), KATA_SCAN or KATA_INTER_AUTO.  In the sequential form
    s_init/z_init give the state before the first token and s_pre/z_pre receive the state after the last."""
    return _call(KATA_FN_CHUNKED, q, k, v, out, C, **kw)


def kata_chunk_state_scan(q, k, v, out=None, C: int = 64, **kw):
    """Chunk-state -> log-depth scan -> chunk-output pipeline; optional s_pre/z_pre export."""
    return _call(KATA_FN_CHUNK_STATE_SCAN, q, k, v, out, C, **kw)


def kata_fwd_host(fn: int, q, k, v, out, C: int = 64, **kw):
    """Same as entry point ``fn`` with (pinned) host tensors; copies ride the current CUDA stream."""
    return _call(fn, q, k, v, out, C, host_io=True, **kw)


def decode_n_psi(d_k: int, feature_order: int = 2, state_layout: int = KATA_LAYOUT_DIRECT, feature_groups: int = 0) -> int:
    """Feature rows of the state: d_k (order 1); g m^2 (direct) or g m(m+1)/2 (packed) with m = d_k / g for the
    PSD lift in g blocks (g = 1: the full lift)."""
    if feature_order == 1:
        return d_k
    g = max(1, feature_groups)
    m = d_k // g
    return g * (m * (m + 1) // 2 if state_layout == KATA_LAYOUT_PACKED else m * m)


def kata_decode_step(q, k, v, S, Z, out=None, *, workspace: Optional[Workspace] = None, stream=None, **opt_kw):
    """One decode token per (b,h): q,k [B,H,d_k], v [B,H,d_v]; fp32 state S [B,H,n_psi,d_v], Z [B,H,n_psi] is
    updated in place.  Returns out [B,H,d_v]."""
    import torch
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and S.is_contiguous() and Z.is_contiguous()):
        raise ValueError("q, k, v, S, Z must be contiguous")
    if S.dtype != torch.float32 or Z.dtype != torch.float32:
        raise ValueError("the state is fp32")
    if out is None:
        out = torch.empty_like(v)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    opts = make_opts(_dtype_code(q), stream=stream, **opt_kw)
    n_psi = decode_n_psi(d_k, opts.feature_order, opts.state_layout, opts.feature_groups)
    if tuple(S.shape) != (B, H, n_psi, d_v) or tuple(Z.shape) != (B, H, n_psi):
        raise ValueError(f"state shapes must be {(B, H, n_psi, d_v)} and {(B, H, n_psi)}")
    need = kata_workspace_bytes(KATA_FN_DECODE_STEP, B, H, 1, d_k, d_v, 0, opts)
    ws = workspace if workspace is not None else _default_ws
    ptr, size = ws.get(need, q.device)
    opts.workspace, opts.workspace_bytes = ptr or None, size
    st = lib().kata_decode_step(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), S.data_ptr(), Z.data_ptr(),
                                B, H, d_k, d_v, ctypes.byref(opts))
    if st != 0:
        raise KataError(st, "kata_decode_step")
    return out


def kata_bwd_quadratic(q, k, v, dout, dq=None, dk=None, dv=None, *, workspace: Optional[Workspace] = None,
                       stream=None, **opt_kw):
    """Gradients of sum(dout * out) with respect to q, k, v (q,k [B,H,T,d_k]; v,dout [B,H,T,d_v]); the forward
    is recomputed.  Returns (dq, dk, dv) in the dtype of the inputs."""
    import torch
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and dout.is_contiguous()):
        raise ValueError("q, k, v, dout must be contiguous [B,H,T,d]")
    B, H, T, d_k = q.shape
    d_v = v.shape[-1]
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    opts = make_opts(_dtype_code(q), stream=stream, **opt_kw)
    need = kata_workspace_bytes(KATA_FN_BWD_QUADRATIC, B, H, T, d_k, d_v, 0, opts)
    ws = workspace if workspace is not None else _default_ws
    ptr, size = ws.get(need, q.device)
    opts.workspace, opts.workspace_bytes = ptr or None, size
    st = lib().kata_bwd_quadratic(q.data_ptr(), k.data_ptr(), v.data_ptr(), dout.data_ptr(), dq.data_ptr(),
                                  dk.data_ptr(), dv.data_ptr(), B, H, T, d_k, d_v, ctypes.byref(opts))
    if st != 0:
        raise KataError(st, "kata_bwd_quadratic")
    return dq, dk, dv


def kata_bwd_chunked(q, k, v, dout, dq=None, dk=None, dv=None, C: int = 64, *, workspace: Optional[Workspace] = None,
                     stream=None, **opt_kw):
    """The same gradients as ``kata_bwd_quadratic`` by the O(T) two-pass linear-state backward.  Returns (dq, dk, dv)
    in the dtype of the inputs."""
    import torch
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and dout.is_contiguous()):
        raise ValueError("q, k, v, dout must be contiguous [B,H,T,d]")
    B, H, T, d_k = q.shape
    d_v = v.shape[-1]
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    opts = make_opts(_dtype_code(q), stream=stream, **opt_kw)
    need = kata_workspace_bytes(KATA_FN_BWD_CHUNKED, B, H, T, d_k, d_v, C, opts)
    ws = workspace if workspace is not None else _default_ws
    ptr, size = ws.get(need, q.device)
    opts.workspace, opts.workspace_bytes = ptr or None, size
    st = lib().kata_bwd_chunked(q.data_ptr(), k.data_ptr(), v.data_ptr(), dout.data_ptr(), dq.data_ptr(),
                                dk.data_ptr(), dv.data_ptr(), B, H, T, d_k, d_v, C, ctypes.byref(opts))
    if st != 0:
        raise KataError(st, "kata_bwd_chunked")
    return dq, dk, dv


KATA_STATIC_SCRATCH_BYTES = 32 << 20


def kata_chunk_state_scan_static(q, k, v, out, C: int = 64, *, scan_group: int = 0, impl: int = KATA_IMPL_AUTO,
                                 feature_order: int = 2, stream=None):
    """The scan pipeline with the library's built-in scratch: for callers that must not allocate.

    Unlike the other wrappers this one never touches torch's allocator: ``out`` must be passed in, and
    no workspace is requested.  Calls that overlap on the GPU share (and race on) the one scratch array.
    """
    import torch
    B, H, T, d_k = q.shape
    d_v = v.shape[-1]
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    opts = make_opts(_dtype_code(q), stream=stream, scan_group=scan_group, impl=impl, feature_order=feature_order)
    st = lib().kata_chunk_state_scan_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), B, H, T, d_k, d_v,
                                            C, ctypes.byref(opts))
    if st != 0:
        raise KataError(st, "kata_chunk_state_scan_static")
    return out
