"""CPU oracle for the GKA hot path: ctypes front end of ``gka_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the product path.  It shares no code with
the CUDA library.  All arithmetic lives in the C file (fp64, token by token,
following eq. (CH), Algorithm 1 and the eigenvalue bounds of Section 4.1); this
module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gka_oracle.c")
_LIB = os.path.join(_HERE, "libgka_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, fp64).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=x86-64-v3", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.check_call(cmd)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        ci = ctypes.c_int
        cd = ctypes.c_double
        lib.gka_oracle_omega.argtypes = [cd, cd, ci, dp]
        lib.gka_oracle_omega.restype = None
        lib.gka_oracle_chebyshev.argtypes = [ci, dp, dp, cd, cd, ci, dp]
        lib.gka_oracle_chebyshev.restype = None
        lib.gka_oracle_cholesky_solve.argtypes = [ci, dp, dp, dp]
        lib.gka_oracle_cholesky_solve.restype = ci
        lib.gka_oracle_fwd.argtypes = [ci] * 5 + [dp] * 7 + [ci, ci] + [dp] * 6 + [ci]
        lib.gka_oracle_fwd.restype = ci
        lib.gka_oracle_decode.argtypes = [ci] * 4 + [dp] * 8 + [ci, ci] + [dp, dp] + [ci]
        lib.gka_oracle_decode.restype = ci
        lib.gka_oracle_max_threads.argtypes = []
        lib.gka_oracle_max_threads.restype = ci
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.POINTER(ctypes.c_double)()
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def max_threads() -> int:
    return int(_load().gka_oracle_max_threads())


def omega_schedule(L: float, mu: float, r: int) -> np.ndarray:
    """omega_0 .. omega_r of Algorithm 1."""
    out = np.zeros(r + 1)
    _load().gka_oracle_omega(float(L), float(mu), int(r), _p(out))
    return out


def chebyshev(A, q, L: float, mu: float, r: int) -> np.ndarray:
    """xi_r of Algorithm 1 for the dense symmetric matrix A."""
    A = _f64(A)
    q = _f64(q)
    D = q.shape[0]
    assert A.shape == (D, D)
    xi = np.zeros(D)
    _load().gka_oracle_chebyshev(D, _p(A), _p(q), float(L), float(mu), int(r), _p(xi))
    return xi


def cholesky_solve(A, b) -> np.ndarray:
    A = _f64(A)
    b = _f64(b)
    x = np.zeros_like(b)
    rc = _load().gka_oracle_cholesky_solve(b.shape[0], _p(A), _p(b), _p(x))
    if rc:
        raise np.linalg.LinAlgError("matrix is not positive definite")
    return x


def fwd(q, k, v, gate, lam, n_iter: int, state_in=None, lam_mode: int = 0, exact: bool = False,
        want_x: bool = False, threads: int = 0, beta=None, alpha=None) -> dict:
    """Token-by-token forward recurrence.

    q, k: [B,T,heads,d_k]; v: [B,T,heads,d_v]; gate, lam, beta (optional write strength), alpha (optional
    alpha-connection: the read uses alpha x + (1 - alpha) q): [B,T,heads].
    Returns dict(out [B,T,heads,d_v], fro [B,T,heads], state [B,heads,d_k*d_k+d_v*d_k],
    and, on request, out_exact and x).
    """
    q, k, v, gate, lam = map(_f64, (q, k, v, gate, lam))
    B, T, Hh, dk = q.shape
    dv = v.shape[-1]
    assert k.shape == q.shape and v.shape[:3] == q.shape[:3]
    assert gate.shape == (B, T, Hh) and lam.shape == (B, T, Hh)
    st = dk * dk + dv * dk
    s_in = None if state_in is None else _f64(state_in).reshape(B, Hh, st)
    out = np.zeros((B, T, Hh, dv))
    out_exact = np.zeros((B, T, Hh, dv)) if exact else None
    fro = np.zeros((B, T, Hh))
    x = np.zeros((B, T, Hh, dk)) if want_x else None
    state = np.zeros((B, Hh, st))
    bt = None if beta is None else _f64(beta)
    assert bt is None or bt.shape == (B, T, Hh)
    al = None if alpha is None else _f64(alpha)
    assert al is None or al.shape == (B, T, Hh)
    rc = _load().gka_oracle_fwd(B, T, Hh, dk, dv, _p(q), _p(k), _p(v), _p(gate), _p(lam), _p(bt), _p(al),
                                int(lam_mode), int(n_iter), _p(s_in), _p(out), _p(out_exact),
                                _p(fro), _p(x), _p(state), int(threads))
    if rc:
        raise np.linalg.LinAlgError("Cholesky failed in the exact branch")
    res = dict(out=out, fro=fro, state=state)
    if exact:
        res["out_exact"] = out_exact
    if want_x:
        res["x"] = x
    return res


def decode(state, q, k, v, gate, lam, n_iter: int, lam_mode: int = 0, exact: bool = False,
           threads: int = 0, beta=None, alpha=None) -> dict:
    """One recurrent step.  state [N,heads,st] is copied, the new state is returned."""
    q, k, v, gate, lam = map(_f64, (q, k, v, gate, lam))
    N, Hh, dk = q.shape
    dv = v.shape[-1]
    st = dk * dk + dv * dk
    new_state = np.array(state, dtype=np.float64, order="C", copy=True).reshape(N, Hh, st)
    out = np.zeros((N, Hh, dv))
    out_exact = np.zeros((N, Hh, dv)) if exact else None
    bt = None if beta is None else _f64(beta)
    al = None if alpha is None else _f64(alpha)
    rc = _load().gka_oracle_decode(N, Hh, dk, dv, _p(new_state), _p(q), _p(k), _p(v), _p(gate),
                                   _p(lam), _p(bt), _p(al), int(lam_mode), int(n_iter), _p(out), _p(out_exact),
                                   int(threads))
    if rc:
        raise np.linalg.LinAlgError("Cholesky failed in the exact branch")
    res = dict(out=out, state=new_state)
    if exact:
        res["out_exact"] = out_exact
    return res
