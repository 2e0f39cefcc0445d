"""Python binding of the C-ABI in include/s2a.h (ctypes; argument marshalling only).

torch is used for device memory and streams.  Every step of the operator runs in the CUDA
library; there is no fallback: if libs2a.so is missing or a call fails, an exception is raised.
Operation: S2-Attn, Algorithm 1 / Section 3.2 of the LongLoRA paper (see include/s2a.h).
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libs2a.so")

S2A_OK = 0
S2A_ERR_INVALID_ARG = -1
S2A_ERR_UNSUPPORTED = -2
S2A_ERR_CUDA = -3
S2A_ERR_TIMEOUT = -4
S2A_ERR_TOO_LARGE = -5

EXPORTS = [
    "s2a_fwd", "s2a_bwd", "s2a_bwd_workspace_bytes", "s2a_bwd_workspace_bytes_fast", "s2a_fwd_ex", "s2a_bwd_ex", "s2a_bwd_stage", "s2a_fwd_bwd_host",
    "s2a_bwd_noalloc", "s2a_bwd_noalloc_max_rows", "s2a_fwd_packed", "s2a_bwd_packed",
    "s2a_selftest_wait_expiry", "s2a_device_status", "s2a_status_string", "s2a_last_cuda_error", "s2a_version",
]

_lib = None


class S2AError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status}, cuda error {last_cuda_error()})")


def load() -> ctypes.CDLL:
    """Load libs2a.so (built by paper_2309_12307_b200/build.py).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2309_12307_b200.build` (needs nvcc)")
    lib = ctypes.CDLL(LIB_PATH)
    P, I, F, Z = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.s2a_fwd.argtypes = [P, P, P, P, P, I, I, I, I, I, I, P]
    lib.s2a_fwd.restype = I
    lib.s2a_bwd.argtypes = [P, P, P, P, P, P, P, P, P, I, I, I, I, I, I, P, Z, P]
    lib.s2a_bwd.restype = I
    lib.s2a_fwd_ex.argtypes = [P, P, P, P, P, I, I, I, I, I, I, F, I, I, ctypes.c_uint, P]
    lib.s2a_fwd_ex.restype = I
    lib.s2a_bwd_ex.argtypes = [P, P, P, P, P, P, P, P, P, I, I, I, I, I, I, F, I, I, ctypes.c_uint, P, Z, P]
    lib.s2a_bwd_ex.restype = I
    lib.s2a_bwd_stage.argtypes = [P, P, P, P, P, P, P, P, P, I, I, I, I, I, I, P, Z, I, P]
    lib.s2a_bwd_stage.restype = I
    lib.s2a_bwd_noalloc.argtypes = [P, P, P, P, P, P, P, P, P, I, I, I, I, I, I, P]
    lib.s2a_bwd_noalloc.restype = I
    lib.s2a_bwd_noalloc_max_rows.restype = Z
    lib.s2a_fwd_packed.argtypes = [P, P, P, I, I, I, I, I, P]
    lib.s2a_fwd_packed.restype = I
    lib.s2a_bwd_packed.argtypes = [P, P, P, P, P, I, I, I, I, I, P, Z, P]
    lib.s2a_bwd_packed.restype = I
    lib.s2a_bwd_workspace_bytes.argtypes = [I, I, I, I, I, I]
    lib.s2a_bwd_workspace_bytes.restype = Z
    lib.s2a_bwd_workspace_bytes_fast.argtypes = [I, I, I, I, I, I, Z]
    lib.s2a_bwd_workspace_bytes_fast.restype = Z
    lib.s2a_fwd_bwd_host.argtypes = [P] * 18 + [I] * 6 + [P, Z, P]
    lib.s2a_fwd_bwd_host.restype = I
    lib.s2a_selftest_wait_expiry.argtypes = [ctypes.c_longlong, P]
    lib.s2a_selftest_wait_expiry.restype = I
    lib.s2a_device_status.argtypes = [ctypes.POINTER(I)]
    lib.s2a_device_status.restype = I
    lib.s2a_status_string.argtypes = [I]
    lib.s2a_status_string.restype = ctypes.c_char_p
    lib.s2a_last_cuda_error.restype = I
    lib.s2a_version.restype = I
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().s2a_status_string(int(status)).decode()


def last_cuda_error() -> int:
    return int(load().s2a_last_cuda_error())


def version() -> int:
    return int(load().s2a_version())


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _check(rc: int, what: str) -> None:
    if rc != S2A_OK:
        raise S2AError(rc, what)


def _require(t, dtype, name: str, shape=None, device=None, cuda: bool = True):
    """One tensor the library will read or write through its raw pointer: it must be what the C side
    takes it for, or the kernels would reinterpret foreign memory."""
    if not isinstance(t, torch.Tensor):
        raise ValueError(f"{name} must be a torch.Tensor")
    if t.is_cuda != cuda:
        raise ValueError(f"{name} must be a {'CUDA' if cuda else 'CPU (pinned)'} tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, not {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, not {tuple(t.shape)}")
    if device is not None and t.device != device:
        raise ValueError(f"{name} must be on {device}, not {t.device}")


def _dims(q, k, v, cuda: bool = True):
    """Checks q [B,N,H,d] and k, v [B,N,Hkv,d] (bf16, contiguous, one device) and returns the sizes."""
    _require(q, torch.bfloat16, "q", cuda=cuda)
    if q.dim() != 4:
        raise ValueError(f"q must be [B, N, H, d], not {tuple(q.shape)}")
    B, N, H, d = q.shape
    _require(k, torch.bfloat16, "k", device=q.device, cuda=cuda)
    if k.dim() != 4 or k.shape[0] != B or k.shape[1] != N or k.shape[3] != d:
        raise ValueError(f"k must be [B, N, Hkv, d] = [{B}, {N}, Hkv, {d}], not {tuple(k.shape)}")
    Hkv = k.shape[2]
    _require(v, torch.bfloat16, "v", shape=k.shape, device=q.device, cuda=cuda)
    return B, N, H, Hkv, d


def _check_fwd_out(q, o, lse):
    B, N, H, d = q.shape
    _require(o, torch.bfloat16, "o", shape=q.shape, device=q.device)
    _require(lse, torch.float32, "lse", shape=(B, H, N), device=q.device)


def _check_bwd(q, k, o, lse, dO, dq, dk, dv):
    _check_fwd_out(q, o, lse)
    _require(dO, torch.bfloat16, "dO", shape=q.shape, device=q.device)
    _require(dq, torch.bfloat16, "dq", shape=q.shape, device=q.device)
    _require(dk, torch.bfloat16, "dk", shape=k.shape, device=q.device)
    _require(dv, torch.bfloat16, "dv", shape=k.shape, device=q.device)


def _check_workspace(ws, device):
    """The workspace's size is checked by the library (S2A_ERR_INVALID_ARG); here only what it is."""
    _require(ws, torch.uint8, "workspace", device=device)


def bwd_workspace_bytes(B, N, H, Hkv, d, G) -> int:
    """Least workspace of the backward (dq then recomputes the scores)."""
    return int(load().s2a_bwd_workspace_bytes(B, N, H, Hkv, d, G))


def bwd_workspace_bytes_fast(B, N, H, Hkv, d, G, budget: int) -> int:
    """Workspace, at most `budget` bytes, with which the backward is fastest (room for spilled dS)."""
    return int(load().s2a_bwd_workspace_bytes_fast(B, N, H, Hkv, d, G, int(budget)))


def _default_workspace(B, N, H, Hkv, d, G, device, fast=True):
    """Workspace for a call that was given none: the fast size within half of the free device memory,
    or the minimum with fast=False."""
    need = bwd_workspace_bytes(B, N, H, Hkv, d, G)
    if fast:
        free, _ = torch.cuda.mem_get_info(device)
        need = max(need, bwd_workspace_bytes_fast(B, N, H, Hkv, d, G, free // 2))
    return torch.empty(max(need, 256), dtype=torch.uint8, device=device)


def s2a_fwd(q, k, v, G, o=None, lse=None, stream=None):
    """o [B,N,H,d] bf16 and lse [B,H,N] fp32 of S2-Attn (second half of the heads shifted by G/2)."""
    B, N, H, Hkv, d = _dims(q, k, v)
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    _check_fwd_out(q, o, lse)
    rc = load().s2a_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), B, N, H, Hkv, d, G,
                        _stream_ptr(stream))
    _check(rc, "s2a_fwd")
    return o, lse


def s2a_bwd(q, k, v, o, lse, dO, G, dq=None, dk=None, dv=None, workspace=None, stream=None, fast=True):
    """dq, dk, dv (bf16) of sum(o * dO).  Without a workspace one is allocated: large enough for the
    spilling backward (fast=True) or the minimum (fast=False: dq recomputes the scores)."""
    B, N, H, Hkv, d = _dims(q, k, v)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    _check_bwd(q, k, o, lse, dO, dq, dk, dv)
    if workspace is None:
        workspace = _default_workspace(B, N, H, Hkv, d, G, q.device, fast)
    _check_workspace(workspace, q.device)
    rc = load().s2a_bwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), dO.data_ptr(),
                        dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), B, N, H, Hkv, d, G, workspace.data_ptr(),
                        workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "s2a_bwd")
    return dq, dk, dv


def bwd_noalloc_max_rows() -> int:
    return int(load().s2a_bwd_noalloc_max_rows())


def s2a_bwd_noalloc(q, k, v, o, lse, dO, G, dq, dk, dv, stream=None):
    """s2a_bwd for callers that cannot supply scratch: D lives in a 4 MiB array inside the library.

    Outputs are written into the dq, dk, dv tensors the caller passes; this wrapper creates no
    tensor.  B*H*N must not exceed bwd_noalloc_max_rows().  Calls that may overlap on the GPU
    share the array and must be serialised (see include/s2a.h).
    """
    B, N, H, Hkv, d = _dims(q, k, v)
    _check_bwd(q, k, o, lse, dO, dq, dk, dv)
    rc = load().s2a_bwd_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
                                dO.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), B, N, H, Hkv, d, G,
                                _stream_ptr(stream))
    _check(rc, "s2a_bwd_noalloc")
    return dq, dk, dv


def _packed_dims(qkv):
    _require(qkv, torch.bfloat16, "qkv")
    if qkv.dim() != 5 or qkv.shape[2] != 3:
        raise ValueError(f"qkv must be [B, N, 3, H, d], not {tuple(qkv.shape)}")
    B, N, _, H, d = qkv.shape
    return B, N, H, d


def s2a_fwd_packed(qkv, G, o=None, lse=None, stream=None):
    """Forward on a packed qkv tensor [B, N, 3, H, d] (the calling convention of Algorithm 1)."""
    B, N, H, d = _packed_dims(qkv)
    o = torch.empty((B, N, H, d), dtype=torch.bfloat16, device=qkv.device) if o is None else o
    lse = torch.empty((B, H, N), dtype=torch.float32, device=qkv.device) if lse is None else lse
    _require(o, torch.bfloat16, "o", shape=(B, N, H, d), device=qkv.device)
    _require(lse, torch.float32, "lse", shape=(B, H, N), device=qkv.device)
    rc = load().s2a_fwd_packed(qkv.data_ptr(), o.data_ptr(), lse.data_ptr(), B, N, H, d, G, _stream_ptr(stream))
    _check(rc, "s2a_fwd_packed")
    return o, lse


def s2a_bwd_packed(qkv, o, lse, dO, G, dqkv=None, workspace=None, stream=None, fast=True):
    """Backward on a packed qkv tensor; returns dqkv [B, N, 3, H, d]."""
    B, N, H, d = _packed_dims(qkv)
    dqkv = torch.empty_like(qkv) if dqkv is None else dqkv
    _require(dqkv, torch.bfloat16, "dqkv", shape=qkv.shape, device=qkv.device)
    _require(o, torch.bfloat16, "o", shape=(B, N, H, d), device=qkv.device)
    _require(dO, torch.bfloat16, "dO", shape=(B, N, H, d), device=qkv.device)
    _require(lse, torch.float32, "lse", shape=(B, H, N), device=qkv.device)
    if workspace is None:
        workspace = _default_workspace(B, N, H, H, d, G, qkv.device, fast)
    _check_workspace(workspace, qkv.device)
    rc = load().s2a_bwd_packed(qkv.data_ptr(), o.data_ptr(), lse.data_ptr(), dO.data_ptr(), dqkv.data_ptr(), B, N, H, d, G,
                               workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "s2a_bwd_packed")
    return dqkv


def s2a_bwd_stage(q, k, v, o, lse, dO, G, dq, dk, dv, workspace, stage, stream=None):
    """Enqueue one kernel of the backward: 0 = D preprocess, 1 = dk/dv, 2 = dq (profiling aid)."""
    B, N, H, Hkv, d = _dims(q, k, v)
    _check_bwd(q, k, o, lse, dO, dq, dk, dv)
    _check_workspace(workspace, q.device)
    rc = load().s2a_bwd_stage(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), dO.data_ptr(),
                              dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), B, N, H, Hkv, d, G, workspace.data_ptr(),
                              workspace.numel() * workspace.element_size(), int(stage), _stream_ptr(stream))
    _check(rc, "s2a_bwd_stage")


S2A_FLAG_LEAK_FREE = 1
S2A_FLAG_SWAP_WRAPPED = 2


def _flags(leak_free, swap_wrapped) -> int:
    return (S2A_FLAG_LEAK_FREE if leak_free else 0) | (S2A_FLAG_SWAP_WRAPPED if swap_wrapped else 0)


def s2a_fwd_ex(q, k, v, G, scale=None, n_unshifted=None, shift=None, leak_free=False, o=None, lse=None, stream=None,
               swap_wrapped=False):
    """Generalised forward: heads [0, n_unshifted) unshifted, the rest rolled by -shift tokens;
    leak_free=True cuts the wrapped group of the shifted heads at the wrap (Appendix B, variant 2);
    swap_wrapped=True makes its two parts change places (variant 3)."""
    B, N, H, Hkv, d = _dims(q, k, v)
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    n_unshifted = H // 2 if n_unshifted is None else n_unshifted
    shift = G // 2 if shift is None else shift
    o = torch.empty_like(q) if o is None else o
    lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if lse is None else lse
    _check_fwd_out(q, o, lse)
    rc = load().s2a_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), B, N, H, Hkv, d, G,
                           scale, n_unshifted, shift, _flags(leak_free, swap_wrapped), _stream_ptr(stream))
    _check(rc, "s2a_fwd_ex")
    return o, lse


def s2a_bwd_ex(q, k, v, o, lse, dO, G, scale=None, n_unshifted=None, shift=None, leak_free=False, workspace=None,
               stream=None, dq=None, dk=None, dv=None, swap_wrapped=False, fast=True):
    B, N, H, Hkv, d = _dims(q, k, v)
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    n_unshifted = H // 2 if n_unshifted is None else n_unshifted
    shift = G // 2 if shift is None else shift
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    _check_bwd(q, k, o, lse, dO, dq, dk, dv)
    if workspace is None:
        workspace = _default_workspace(B, N, H, Hkv, d, G, q.device, fast)
    _check_workspace(workspace, q.device)
    rc = load().s2a_bwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), dO.data_ptr(),
                           dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), B, N, H, Hkv, d, G, scale, n_unshifted, shift,
                           _flags(leak_free, swap_wrapped), workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "s2a_bwd_ex")
    return dq, dk, dv


def s2a_fwd_bwd_host(host_in, host_out, dev, G, workspace, stream=None):
    """Forward+backward from pinned host tensors.

    host_in  = (q, k, v, dO) CPU bf16 tensors; host_out = (o, lse, dq, dk, dv) CPU tensors to fill;
    dev      = (q, k, v, dO, o, lse, dq, dk, dv) device buffers of the same shapes.
    Work is only enqueued: synchronise the stream before reading host_out.
    """
    hq, hk, hv, hdo = host_in
    ho, hlse, hdq, hdk, hdv = host_out
    B, N, H, Hkv, d = _dims(hq, hk, hv, cuda=False)
    bf, f32 = torch.bfloat16, torch.float32
    for t, name, dt, shp in ((hdo, "host dO", bf, hq.shape), (ho, "host o", bf, hq.shape), (hlse, "host lse", f32, (B, H, N)),
                             (hdq, "host dq", bf, hq.shape), (hdk, "host dk", bf, hk.shape), (hdv, "host dv", bf, hk.shape)):
        _require(t, dt, name, shape=shp, cuda=False)
    if len(dev) != 9:
        raise ValueError("dev must hold the nine device buffers (q, k, v, dO, o, lse, dq, dk, dv)")
    shapes = (hq.shape, hk.shape, hk.shape, hq.shape, hq.shape, (B, H, N), hq.shape, hk.shape, hk.shape)
    for t, shp, name in zip(dev, shapes, ("q", "k", "v", "dO", "o", "lse", "dq", "dk", "dv")):
        _require(t, f32 if name == "lse" else bf, f"device {name}", shape=shp, device=dev[0].device)
    _check_workspace(workspace, dev[0].device)
    ptrs = [t.data_ptr() for t in (hq, hk, hv, hdo, ho, hlse, hdq, hdk, hdv)] + [t.data_ptr() for t in dev]
    rc = load().s2a_fwd_bwd_host(*ptrs, B, N, H, Hkv, d, G, workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "s2a_fwd_bwd_host")


def selftest_wait_expiry(limit_cycles: int = 1_000_000, stream=None) -> None:
    """Enqueue the diagnostic kernel whose bounded wait runs out after `limit_cycles` SM cycles."""
    _check(load().s2a_selftest_wait_expiry(int(limit_cycles), _stream_ptr(stream)), "s2a_selftest_wait_expiry")


def device_status():
    """(status, where): S2A_OK, or S2A_ERR_TIMEOUT with the code of the wait that expired."""
    where = ctypes.c_int(0)
    rc = load().s2a_device_status(ctypes.byref(where))
    return int(rc), int(where.value)
