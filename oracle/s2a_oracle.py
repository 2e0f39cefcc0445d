"""ctypes front end of the CPU fp64 oracle (oracle/s2a_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The GPU package never imports this module.

Inputs may be fp64 tensors/arrays (used as they are) or torch.bfloat16 tensors
(their bits are handed to the C code, which widens them exactly).  All results
are fp64 numpy arrays.  Operation: Algorithm 1 / Section 3.2 / Eq. 1 of the
LongLoRA paper; see the header of s2a_oracle.c for the index form.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "s2a_oracle.c")
_LIB = os.path.join(_HERE, "libs2a_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P, I, LL, D = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_double
        lib.s2a_oracle_fwd_ex.argtypes = [P, P, P, I, I, I, I, I, I, I, D, I, I, I, P, LL, P, P]
        lib.s2a_oracle_fwd_ex.restype = I
        lib.s2a_oracle_bwd_ex.argtypes = [P, P, P, P, I, I, I, I, I, I, I, D, I, I, I, P, LL, P, LL, P, P, P]
        lib.s2a_oracle_bwd_ex.restype = I
        lib.s2a_oracle_attended.argtypes = [I, I, I, I, I, P]
        lib.s2a_oracle_attended.restype = I
        lib.s2a_oracle_num_threads.restype = I
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().s2a_oracle_num_threads())


def _as_input(x):
    """Return (keepalive, pointer, dtype_code) for an fp64 or bf16 input."""
    try:
        import torch
    except ImportError:  # numpy-only callers
        torch = None
    if torch is not None and isinstance(x, torch.Tensor):
        x = x.detach().cpu().contiguous()
        if x.dtype == torch.bfloat16:
            a = x.view(torch.int16).numpy()
            return a, a.ctypes.data, 1
        a = x.to(torch.float64).numpy()
        return a, a.ctypes.data, 0
    a = np.ascontiguousarray(x, dtype=np.float64)
    return a, a.ctypes.data, 0


def _rows(rows):
    if rows is None:
        return None, None, 0
    a = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 3))
    return a, a.ctypes.data, a.shape[0]


def _defaults(H, G, d, scale, n_unshifted, shift):
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    if n_unshifted is None:
        if H % 2:
            raise ValueError("H must be even to split the heads in two halves")
        n_unshifted = H // 2
    if shift is None:
        if G % 2:
            raise ValueError("G must be even to shift by G/2")
        shift = G // 2
    return float(scale), int(n_unshifted), int(shift)


def _variant(leak_free, swap_wrapped) -> int:
    """0 = Algorithm 1, 1 = variant 2 of Appendix B, 2 = variant 3 (they exclude each other)."""
    if leak_free and swap_wrapped:
        raise ValueError("variants 2 and 3 exclude each other")
    return 1 if leak_free else (2 if swap_wrapped else 0)


def fwd(q, k, v, G, scale=None, rows=None, n_unshifted=None, shift=None, leak_free=False, swap_wrapped=False):
    """o, lse.  rows=None: o [B,N,H,d], lse [B,H,N].  rows=[(b,h,t),...]: o [n,d], lse [n].
    leak_free=True is variant 2 of Appendix B: the wrapped group of a shifted head is cut at the wrap.
    swap_wrapped=True is variant 3: the two parts of the wrapped group change places (original token order)."""
    B, N, H, d = q.shape
    Hkv = k.shape[2]
    scale, n_unshifted, shift = _defaults(H, G, d, scale, n_unshifted, shift)
    qa, qp, dt = _as_input(q)
    ka, kp, dtk = _as_input(k)
    va, vp, dtv = _as_input(v)
    assert dt == dtk == dtv, "q, k, v must share a dtype"
    ra, rp, n = _rows(rows)
    if rows is None:
        o = np.empty((B, N, H, d), dtype=np.float64)
        lse = np.empty((B, H, N), dtype=np.float64)
    else:
        o = np.empty((n, d), dtype=np.float64)
        lse = np.empty((n,), dtype=np.float64)
    rc = _load().s2a_oracle_fwd_ex(qp, kp, vp, dt, B, N, H, Hkv, d, G, scale, n_unshifted, shift, _variant(leak_free, swap_wrapped), rp, n,
                                   o.ctypes.data, lse.ctypes.data)
    if rc:
        raise ValueError(f"s2a_oracle_fwd_ex failed ({rc})")
    return o, lse


def bwd(q, k, v, dO, G, scale=None, q_rows=None, kv_rows=None, n_unshifted=None, shift=None, leak_free=False,
        swap_wrapped=False):
    """dq, dk, dv.  With row lists: dq [n_q,d] for (b,h,t) rows, dk/dv [n_kv,d] for (b,hkv,t) rows."""
    B, N, H, d = q.shape
    Hkv = k.shape[2]
    scale, n_unshifted, shift = _defaults(H, G, d, scale, n_unshifted, shift)
    qa, qp, dt = _as_input(q)
    ka, kp, dt1 = _as_input(k)
    va, vp, dt2 = _as_input(v)
    da, dp, dt3 = _as_input(dO)
    assert dt == dt1 == dt2 == dt3, "q, k, v, dO must share a dtype"
    qa_, qrp, nq = _rows(q_rows)
    ka_, krp, nkv = _rows(kv_rows)
    dq = np.empty((B, N, H, d) if q_rows is None else (max(nq, 1), d), dtype=np.float64)
    dk = np.empty((B, N, Hkv, d) if kv_rows is None else (max(nkv, 1), d), dtype=np.float64)
    dv = np.empty_like(dk)
    # an empty list must still be a non-NULL pointer ("skip this part"), NULL means "all rows"
    dummy = np.zeros(3, dtype=np.int32)
    if q_rows is not None and nq == 0:
        qrp = dummy.ctypes.data
    if kv_rows is not None and nkv == 0:
        krp = dummy.ctypes.data
    rc = _load().s2a_oracle_bwd_ex(qp, kp, vp, dp, dt, B, N, H, Hkv, d, G, scale, n_unshifted, shift, _variant(leak_free, swap_wrapped),
                                   qrp, nq,
                                   krp, nkv, dq.ctypes.data, dk.ctypes.data, dv.ctypes.data)
    if rc:
        raise ValueError(f"s2a_oracle_bwd_ex failed ({rc})")
    if q_rows is not None:
        dq = dq[:nq]
    if kv_rows is not None:
        dk, dv = dk[:nkv], dv[:nkv]
    return dq, dk, dv


def attended(N, H, G, h, t):
    """Original-token ids that (head h, token t) attends, in rolled order."""
    out = np.empty(G, dtype=np.int32)
    n = _load().s2a_oracle_attended(N, H, G, h, t, out.ctypes.data)
    if n < 0:
        raise ValueError("bad arguments")
    return out[:n].tolist()
