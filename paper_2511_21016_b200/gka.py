"""Thin ctypes binding of the GKA C ABI (include/gka.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
``libgka.so``.  PyTorch is used for device memory and streams.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgka.so")

GKA_OK = 0
GKA_F32, GKA_BF16 = 0, 1
GKA_PREC_NATIVE, GKA_PREC_HIGH = 0, 1
GKA_FLAG_ADAPTIVE_LAMBDA = 1
GKA_FLAG_VALIDATE = 2
GKA_ERR_TIMEOUT = 8

EXPORTS = ("gka_fwd_workspace_bytes", "gka_fwd_chunked", "gka_decode_step", "gka_status_string",
           "gka_fwd_num_work_items", "gka_fwd_work_range", "gka_last_error_detail",
           "gka_fwd_chunked_noalloc", "gka_noalloc_scratch_bytes", "gka_selftest_bounded_wait",
           "gka_fwd_chunked_host", "gka_fwd_host_staging_bytes", "gka_solve_chunked", "gka_decode_tokens")


class GkaDesc(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int), ("T", ctypes.c_int), ("heads", ctypes.c_int),
        ("d_k", ctypes.c_int), ("d_v", ctypes.c_int),
        ("io_dtype", ctypes.c_int), ("precision", ctypes.c_int), ("flags", ctypes.c_uint),
        ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("state_in", ctypes.c_void_p),
        ("device_status", ctypes.c_void_p), ("fro_out", ctypes.c_void_p),
        ("profile_start", ctypes.c_void_p), ("profile_stop", ctypes.c_void_p), ("beta", ctypes.c_void_p),
        ("alpha", ctypes.c_void_p),
    ]


class GkaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == 7:
            detail = " [" + load_library().gka_last_error_detail().decode() + "]"
        super().__init__(f"{where}: {status_string(status)}{detail}")


_lib = None


def load_library():
    """Load libgka.so (built in-tree by ``build.build_library``).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2511_21016_b200.build` "
                "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        dp = ctypes.POINTER(GkaDesc)
        lib.gka_fwd_workspace_bytes.argtypes = [dp, ci]
        lib.gka_fwd_workspace_bytes.restype = ctypes.c_size_t
        lib.gka_fwd_num_work_items.argtypes = [dp, ci]
        lib.gka_fwd_num_work_items.restype = ci
        lib.gka_fwd_chunked.argtypes = [dp, vp, vp, vp, vp, vp, ci, ci, vp, vp]
        lib.gka_fwd_chunked.restype = ci
        lib.gka_fwd_chunked_noalloc.argtypes = [dp, vp, vp, vp, vp, vp, ci, ci, vp, vp]
        lib.gka_fwd_chunked_noalloc.restype = ci
        lib.gka_noalloc_scratch_bytes.argtypes = []
        lib.gka_noalloc_scratch_bytes.restype = ctypes.c_size_t
        lib.gka_fwd_host_staging_bytes.argtypes = [dp]
        lib.gka_fwd_host_staging_bytes.restype = ctypes.c_size_t
        lib.gka_fwd_chunked_host.argtypes = [dp, vp, vp, vp, vp, vp, vp, ci, ci, vp, vp]
        lib.gka_fwd_chunked_host.restype = ci
        lib.gka_solve_chunked.argtypes = [dp, vp, vp, vp, vp, ci, ci, vp]
        lib.gka_solve_chunked.restype = ci
        lib.gka_decode_step.argtypes = [dp, vp, vp, vp, vp, vp, vp, ci, vp]
        lib.gka_decode_step.restype = ci
        lib.gka_decode_tokens.argtypes = [dp, vp, vp, vp, vp, vp, vp, ci, vp]
        lib.gka_decode_tokens.restype = ci
        llp, ip = ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(ctypes.c_int)
        lib.gka_fwd_work_range.argtypes = [dp, ci, ci, ci, llp, llp, ip, ip]
        lib.gka_fwd_work_range.restype = ci
        lib.gka_last_error_detail.argtypes = []
        lib.gka_last_error_detail.restype = ctypes.c_char_p
        lib.gka_selftest_bounded_wait.argtypes = [dp, ci]
        lib.gka_selftest_bounded_wait.restype = ci
        lib.gka_status_string.argtypes = [ci]
        lib.gka_status_string.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().gka_status_string(int(status)).decode()


def _io_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GKA_F32
    if t.dtype == torch.bfloat16:
        return GKA_BF16
    raise TypeError(f"unsupported I/O dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check_cuda(*ts):
    for t in ts:
        if t is not None:
            if not t.is_cuda:
                raise ValueError("all tensors must live on the CUDA device (no CPU fallback)")
            if not t.is_contiguous():
                raise ValueError("tensors must be contiguous")


def _expect(name, t, dtype, shape):
    """Raise ValueError unless tensor ``t`` (None is allowed: an optional argument) has this dtype and shape.
    The kernels trust the descriptor: a tensor of another size or type would be read or written out of bounds."""
    if t is None:
        return
    if t.dtype != dtype:
        raise ValueError(f"{name}: dtype {t.dtype}, expected {dtype}")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: shape {tuple(t.shape)}, expected {tuple(shape)}")


def _expect_tokens(q, k, v, gate, lam, out, names=("q", "k", "v", "out"), **scalars):
    """q, k, v, out: one I/O dtype and shape [.., heads, d]; gate, lam and the other per-token scalars: float32 [.., heads]."""
    if q.dim() < 3:
        raise ValueError(f"{names[0]}: expected [..., heads, d], got shape {tuple(q.shape)}")
    _io_code(q)
    for n, t in zip(names[1:], (k, v, out)):
        _expect(n, t, q.dtype, q.shape)
    for n, t in dict(gate=gate, lam=lam, **scalars).items():
        _expect(n, t, torch.float32, q.shape[:-1])


def make_desc(B, T, heads, d_k, d_v, io_dtype, precision=GKA_PREC_NATIVE, flags=0, stream=None,
              workspace=None, state_in=None, device_status=None, fro_out=None,
              profile_events=None, beta=None, alpha=None) -> GkaDesc:
    d = GkaDesc()
    d.B, d.T, d.heads, d.d_k, d.d_v = B, T, heads, d_k, d_v
    d.io_dtype, d.precision, d.flags = io_dtype, precision, flags
    d.stream = stream
    d.workspace = _ptr(workspace)
    d.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    d.state_in = _ptr(state_in)
    d.device_status = _ptr(device_status)
    d.fro_out = _ptr(fro_out)
    d.beta = _ptr(beta)
    d.alpha = _ptr(alpha)
    if profile_events is not None:
        d.profile_start, d.profile_stop = profile_events
    return d


def gka_fwd_workspace_bytes(B, T, heads, d, io_dtype=GKA_BF16, chunk=64) -> int:
    desc = make_desc(B, T, heads, d, d, io_dtype)
    return int(load_library().gka_fwd_workspace_bytes(ctypes.byref(desc), chunk))


def gka_fwd_num_work_items(B, T, heads, d, io_dtype=GKA_BF16, chunk=64) -> int:
    desc = make_desc(B, T, heads, d, d, io_dtype)
    return int(load_library().gka_fwd_num_work_items(ctypes.byref(desc), chunk))


def gka_fwd_work_range(B, T, heads, d, num_items, item, chunk=64, io_dtype=GKA_BF16):
    """(first_chunk, end_chunk, cut_in, cut_out) of one work item; host arithmetic only."""
    desc = make_desc(B, T, heads, d, d, io_dtype)
    lo, hi = ctypes.c_longlong(), ctypes.c_longlong()
    ci_, co_ = ctypes.c_int(), ctypes.c_int()
    rc = load_library().gka_fwd_work_range(ctypes.byref(desc), chunk, num_items, item,
                                           ctypes.byref(lo), ctypes.byref(hi), ctypes.byref(ci_),
                                           ctypes.byref(co_))
    if rc != GKA_OK:
        raise GkaError(rc, "gka_fwd_work_range")
    return lo.value, hi.value, bool(ci_.value), bool(co_.value)


def alloc_workspace(B, T, heads, d, device, chunk=64, io_dtype=GKA_BF16, precision=GKA_PREC_NATIVE) -> torch.Tensor:
    desc = make_desc(B, T, heads, d, d, io_dtype, precision)
    n = int(load_library().gka_fwd_workspace_bytes(ctypes.byref(desc), chunk))
    if n == 0:
        raise GkaError(2, "gka_fwd_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def gka_fwd_chunked(q, k, v, gate, lam, n_iter, chunk=64, out=None, state_out=None, *,
                    state_in=None, workspace=None, precision=GKA_PREC_NATIVE, flags=0,
                    fro_out=None, device_status=None, stream=None, profile_events=None, beta=None, alpha=None):
    """Chunk-wise GKA forward.  q,k,v: [B,T,heads,d] (f32 or bf16); gate, lam, beta (optional): [B,T,heads] f32.

    Returns (out, state_out).  Work is enqueued on ``stream`` (default: torch's current stream).
    """
    if q.dim() != 4:
        raise ValueError(f"q: expected [B, T, heads, d], got shape {tuple(q.shape)}")
    B, T, heads, d = q.shape
    _expect_tokens(q, k, v, gate, lam, out, fro_out=fro_out, beta=beta, alpha=alpha)
    _expect("state_out", state_out, torch.float32, (B, heads, 2 * d * d))
    _expect("state_in", state_in, torch.float32, (B, heads, 2 * d * d))
    _expect("device_status", device_status, torch.int32, (1,))
    _check_cuda(q, k, v, gate, lam, out, state_out, state_in, workspace, fro_out, device_status, beta, alpha)
    if out is None:
        out = torch.empty_like(v)
    if state_out is None:
        state_out = torch.empty(B, heads, 2 * d * d, dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(B, T, heads, d, q.device, chunk, _io_code(q), precision)
    elif workspace.dtype != torch.uint8:
        raise ValueError("workspace: expected a uint8 tensor")
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    desc = make_desc(B, T, heads, d, v.shape[-1], _io_code(q), precision, flags, stream, workspace,
                     state_in, device_status, fro_out, profile_events, beta, alpha)
    rc = load_library().gka_fwd_chunked(ctypes.byref(desc), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                        gate.data_ptr(), lam.data_ptr(), int(n_iter), int(chunk),
                                        out.data_ptr(), _ptr(state_out))
    if rc != GKA_OK:
        raise GkaError(rc, "gka_fwd_chunked")
    return out, state_out


def gka_solve_chunked(rhs, k, gate, lam, n_iter, chunk=64, out=None, *, state_in=None, workspace=None,
                      precision=GKA_PREC_NATIVE, flags=0, device_status=None, stream=None, beta=None):
    """The solve alone: x_t = CH(H_t + lambda_t I, rhs_t, n_iter).  rhs, k: [B,T,heads,d]; gate, lam: [B,T,heads] f32.

    With rhs = q this is the iterate the forward multiplies by U_t; with rhs = dL/dx it is dL/dq.
    """
    if rhs.dim() != 4:
        raise ValueError(f"rhs: expected [B, T, heads, d], got shape {tuple(rhs.shape)}")
    B, T, heads, d = rhs.shape
    _expect_tokens(rhs, k, None, gate, lam, out, names=("rhs", "k", "v", "x_out"), beta=beta)
    _expect("state_in", state_in, torch.float32, (B, heads, 2 * d * d))
    _expect("device_status", device_status, torch.int32, (1,))
    _check_cuda(rhs, k, gate, lam, out, state_in, workspace, device_status)
    if out is None:
        out = torch.empty_like(rhs)
    if workspace is None:
        workspace = alloc_workspace(B, T, heads, d, rhs.device, chunk, _io_code(rhs), precision)
    if stream is None:
        stream = torch.cuda.current_stream(rhs.device).cuda_stream
    desc = make_desc(B, T, heads, d, d, _io_code(rhs), precision, flags, stream, workspace, state_in, device_status,
                     beta=beta)
    rc = load_library().gka_solve_chunked(ctypes.byref(desc), rhs.data_ptr(), k.data_ptr(), gate.data_ptr(),
                                          lam.data_ptr(), int(n_iter), int(chunk), out.data_ptr())
    if rc != GKA_OK:
        raise GkaError(rc, "gka_solve_chunked")
    return out


def gka_fwd_host_staging_bytes(B, T, heads, d, io_dtype) -> int:
    desc = make_desc(B, T, heads, d, d, io_dtype)
    return int(load_library().gka_fwd_host_staging_bytes(ctypes.byref(desc)))


def gka_fwd_chunked_host(q, k, v, gate, lam, n_iter, chunk, out, state_out, *, staging, workspace,
                         precision=GKA_PREC_NATIVE, flags=0, stream=None, device_status=None):
    """Host-buffer forward: q, k, v, gate, lam, out, state_out are (pinned) CPU tensors; staging and
    workspace are CUDA byte tensors.  Copies and kernels are enqueued on the stream; no synchronisation."""
    if q.dim() != 4:
        raise ValueError(f"q: expected [B, T, heads, d], got shape {tuple(q.shape)}")
    B, T, heads, d = q.shape
    if out is None:
        raise ValueError("out: the host-buffer call writes into a caller-provided CPU tensor")
    _expect_tokens(q, k, v, gate, lam, out)
    _expect("state_out", state_out, torch.float32, (B, heads, 2 * d * d))
    _expect("device_status", device_status, torch.int32, (1,))
    for t in (q, k, v, gate, lam, out, state_out):
        if t is not None and (t.is_cuda or not t.is_contiguous()):
            raise ValueError("host-buffer call takes contiguous CPU tensors")
    _check_cuda(staging, workspace, device_status)
    need = gka_fwd_host_staging_bytes(B, T, heads, d, _io_code(q))
    if staging.dtype != torch.uint8 or staging.numel() < need:
        raise ValueError(f"staging: expected a uint8 tensor of at least {need} bytes")
    if stream is None:
        stream = torch.cuda.current_stream(staging.device).cuda_stream
    desc = make_desc(B, T, heads, d, v.shape[-1], _io_code(q), precision, flags, stream, workspace,
                     device_status=device_status)
    rc = load_library().gka_fwd_chunked_host(ctypes.byref(desc), staging.data_ptr(), q.data_ptr(),
                                             k.data_ptr(), v.data_ptr(), gate.data_ptr(), lam.data_ptr(),
                                             int(n_iter), int(chunk), out.data_ptr(), _ptr(state_out))
    if rc != GKA_OK:
        raise GkaError(rc, "gka_fwd_chunked_host")
    return out, state_out


def gka_fwd_chunked_noalloc(q, k, v, gate, lam, n_iter, chunk=64, out=None, state_out=None, *,
                            state_in=None, precision=GKA_PREC_NATIVE, flags=0, stream=None):
    """Chunk-wise forward for callers that cannot provide scratch memory: the library's built-in
    scratch array is used instead of a workspace.  ``out`` and ``state_out`` must be given by such
    callers; they are only created here (with torch) when omitted, for convenience in tests."""
    if q.dim() != 4:
        raise ValueError(f"q: expected [B, T, heads, d], got shape {tuple(q.shape)}")
    B, T, heads, d = q.shape
    _expect_tokens(q, k, v, gate, lam, out)
    _expect("state_out", state_out, torch.float32, (B, heads, 2 * d * d))
    _expect("state_in", state_in, torch.float32, (B, heads, 2 * d * d))
    _check_cuda(q, k, v, gate, lam, out, state_out, state_in)
    if out is None:
        out = torch.empty_like(v)
    if state_out is None:
        state_out = torch.empty(B, heads, 2 * d * d, dtype=torch.float32, device=q.device)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    desc = make_desc(B, T, heads, d, v.shape[-1], _io_code(q), precision, flags, stream, None, state_in)
    rc = load_library().gka_fwd_chunked_noalloc(ctypes.byref(desc), q.data_ptr(), k.data_ptr(),
                                                v.data_ptr(), gate.data_ptr(), lam.data_ptr(),
                                                int(n_iter), int(chunk), out.data_ptr(),
                                                _ptr(state_out))
    if rc != GKA_OK:
        raise GkaError(rc, "gka_fwd_chunked_noalloc")
    return out, state_out


def gka_decode_step(state, q, k, v, gate, lam, n_iter, out=None, *, flags=0, device_status=None,
                    stream=None, profile_events=None, beta=None, alpha=None):
    """One recurrent step.  state: [N,heads,2*d*d] f32, updated in place; q,k,v: [N,heads,d]."""
    if q.dim() != 3:
        raise ValueError(f"q: expected [N, heads, d], got shape {tuple(q.shape)}")
    N, heads, d = q.shape
    _expect_tokens(q, k, v, gate, lam, out, beta=beta, alpha=alpha)
    _expect("state", state, torch.float32, (N, heads, 2 * d * d))
    _expect("device_status", device_status, torch.int32, (1,))
    _check_cuda(state, q, k, v, gate, lam, out, device_status, beta, alpha)
    if out is None:
        out = torch.empty_like(v)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    desc = make_desc(N, 1, heads, d, v.shape[-1], _io_code(q), GKA_PREC_NATIVE, flags, stream,
                     device_status=device_status, profile_events=profile_events, beta=beta, alpha=alpha)
    rc = load_library().gka_decode_step(ctypes.byref(desc), state.data_ptr(), q.data_ptr(),
                                        k.data_ptr(), v.data_ptr(), gate.data_ptr(), lam.data_ptr(),
                                        int(n_iter), out.data_ptr())
    if rc != GKA_OK:
        raise GkaError(rc, "gka_decode_step")
    return out


def gka_decode_tokens(state, q, k, v, gate, lam, n_iter, out=None, *, flags=0, device_status=None,
                      stream=None, profile_events=None, beta=None, alpha=None):
    """The recurrent step over T consecutive tokens.  state: [N,heads,2*d*d] f32, updated in place;
    q,k,v: [N,T,heads,d]; gate, lam (beta, alpha): [N,T,heads]."""
    if q.dim() != 4:
        raise ValueError(f"q: expected [N, T, heads, d], got shape {tuple(q.shape)}")
    N, T, heads, d = q.shape
    _expect_tokens(q, k, v, gate, lam, out, beta=beta, alpha=alpha)
    _expect("state", state, torch.float32, (N, heads, 2 * d * d))
    _expect("device_status", device_status, torch.int32, (1,))
    _check_cuda(state, q, k, v, gate, lam, out, device_status, beta, alpha)
    if out is None:
        out = torch.empty_like(v)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    desc = make_desc(N, T, heads, d, v.shape[-1], _io_code(q), GKA_PREC_NATIVE, flags, stream,
                     device_status=device_status, profile_events=profile_events, beta=beta, alpha=alpha)
    rc = load_library().gka_decode_tokens(ctypes.byref(desc), state.data_ptr(), q.data_ptr(),
                                          k.data_ptr(), v.data_ptr(), gate.data_ptr(), lam.data_ptr(),
                                          int(n_iter), out.data_ptr())
    if rc != GKA_OK:
        raise GkaError(rc, "gka_decode_tokens")
    return out


def gka_selftest_bounded_wait(device_status, polls=4096, stream=None):
    """Self-test of the bounded device-side waits: a one-block kernel polls an mbarrier that nothing arrives at,
    gives up after ``polls`` polls and stores GKA_ERR_TIMEOUT into ``device_status`` (an int32 CUDA tensor)."""
    _expect("device_status", device_status, torch.int32, (1,))
    _check_cuda(device_status)
    if stream is None:
        stream = torch.cuda.current_stream(device_status.device).cuda_stream
    desc = make_desc(1, 1, 1, 128, 128, GKA_BF16, stream=stream, device_status=device_status)
    rc = load_library().gka_selftest_bounded_wait(ctypes.byref(desc), int(polls))
    if rc != 0:
        raise GkaError(rc, "gka_selftest_bounded_wait")

