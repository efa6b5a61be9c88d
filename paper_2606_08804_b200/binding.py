"""Thin ctypes binding of ``libqdelta.so`` (declared in ``include/qdelta.h``).

Argument marshalling only: torch supplies device memory and the current stream; every step of
the computation runs in the library's CUDA kernels.  There is no fallback: if the library has
not been built, or a call returns an error code, an exception is raised.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqdelta.so")

QD_F32, QD_BF16 = 0, 1
QD_FWD_SAVE_FOR_BWD, QD_BWD_REUSE_FWD, QD_COEF_LOGITS, QD_NORM_QK, QD_STATE_BF16 = 1, 2, 4, 8, 16

EXPORTS = ("qdelta_chunk_workspace_bytes", "qdelta_chunk_fwd", "qdelta_chunk_bwd",
           "qdelta_recurrent_step", "qdelta_workspace_status", "qdelta_status_string",
           "qdelta_profile_enable", "qdelta_profile_stage_count", "qdelta_profile_stage_name",
           "qdelta_profile_read", "qdelta_chunk_fwd_static", "qdelta_chunk_path",
           "qdelta_recurrent_steps")


class QdShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int), ("T", ctypes.c_int), ("H", ctypes.c_int), ("dk", ctypes.c_int),
                ("dv", ctypes.c_int), ("chunk", ctypes.c_int), ("dtype", ctypes.c_int)]


class QdeltaError(RuntimeError):
    pass


_lib = None


def load():
    """Load libqdelta.so (once).  Raises if it is missing: there is no other code path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise QdeltaError("libqdelta.so is not built: run `python -m paper_2606_08804_b200.build` "
                          "(or __graft_entry__.build()); there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, sz, u, i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint, ctypes.c_int
    lib.qdelta_chunk_workspace_bytes.restype = sz
    lib.qdelta_chunk_workspace_bytes.argtypes = [ctypes.POINTER(QdShape), i]
    lib.qdelta_chunk_path.restype = i
    lib.qdelta_chunk_path.argtypes = [ctypes.POINTER(QdShape)]
    lib.qdelta_chunk_fwd.restype = i
    lib.qdelta_chunk_fwd.argtypes = [ctypes.POINTER(QdShape)] + [vp] * 9 + [vp, sz, u, vp]
    lib.qdelta_chunk_bwd.restype = i
    lib.qdelta_chunk_bwd.argtypes = [ctypes.POINTER(QdShape)] + [vp] * 16 + [vp, sz, u, vp]
    lib.qdelta_chunk_fwd_static.restype = i
    lib.qdelta_chunk_fwd_static.argtypes = [ctypes.POINTER(QdShape)] + [vp] * 9 + [vp, vp]
    lib.qdelta_recurrent_step.restype = i
    lib.qdelta_recurrent_step.argtypes = [i] * 5 + [vp] * 8 + [vp]
    lib.qdelta_recurrent_steps.restype = i
    lib.qdelta_recurrent_steps.argtypes = [i] * 6 + [vp] * 8 + [u, vp]
    lib.qdelta_workspace_status.restype = i
    lib.qdelta_workspace_status.argtypes = [vp, ctypes.POINTER(i), vp]
    lib.qdelta_status_string.restype = ctypes.c_char_p
    lib.qdelta_status_string.argtypes = [i]
    lib.qdelta_profile_enable.restype = i
    lib.qdelta_profile_enable.argtypes = [i]
    lib.qdelta_profile_stage_count.restype = i
    lib.qdelta_profile_stage_name.restype = ctypes.c_char_p
    lib.qdelta_profile_stage_name.argtypes = [i]
    lib.qdelta_profile_read.restype = i
    lib.qdelta_profile_read.argtypes = [i, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong), i]
    _lib = lib
    return lib


def profile_enable(on: bool) -> None:
    """Turn the library's per-kernel CUDA-event timing on or off."""
    load().qdelta_profile_enable(1 if on else 0)


def profile_read(reset: bool = True) -> dict:
    """{stage name: (total ms, launches)} of everything recorded since the last reset."""
    lib = load()
    out = {}
    for st in range(lib.qdelta_profile_stage_count()):
        ms, n = ctypes.c_double(0), ctypes.c_longlong(0)
        _check(lib.qdelta_profile_read(st, ctypes.byref(ms), ctypes.byref(n), 1 if reset else 0),
               "qdelta_profile_read")
        out[lib.qdelta_profile_stage_name(st).decode()] = (ms.value, n.value)
    return out


def status_string(code: int) -> str:
    return load().qdelta_status_string(int(code)).decode()


def _check(rc, what):
    if rc != 0:
        raise QdeltaError("%s failed: %s (%d)" % (what, status_string(rc), rc))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return QD_F32
    if t.dtype == torch.bfloat16:
        return QD_BF16
    raise QdeltaError("unsupported dtype %s" % t.dtype)


def _ptr(t, dtype=None, shape=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise QdeltaError("%s must be a contiguous CUDA tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise QdeltaError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise QdeltaError("%s must have shape %s, got %s" % (name, tuple(shape), tuple(t.shape)))
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def make_shape(q, v, chunk) -> QdShape:
    B, T, H, dk = q.shape
    return QdShape(B, T, H, dk, v.shape[-1], int(chunk), _dtype_code(q))


def chunk_workspace_bytes(shape: QdShape, for_backward: bool) -> int:
    n = load().qdelta_chunk_workspace_bytes(ctypes.byref(shape), 1 if for_backward else 0)
    if n == 0:
        raise QdeltaError("unsupported or invalid shape for the chunkwise kernels")
    return int(n)


def chunk_path(shape: QdShape) -> str:
    """Which kernels serve this shape: "tensor_core" (tcgen05) or "fp32" (plain FMA)."""
    r = load().qdelta_chunk_path(ctypes.byref(shape))
    if r < 0:
        raise QdeltaError("unsupported or invalid shape for the chunkwise kernels")
    return "tensor_core" if r == 1 else "fp32"


def alloc_workspace(shape: QdShape, for_backward: bool, device) -> torch.Tensor:
    return torch.empty(chunk_workspace_bytes(shape, for_backward), dtype=torch.uint8, device=device)


def workspace_status(workspace: torch.Tensor) -> int:
    out = ctypes.c_int(0)
    _check(load().qdelta_workspace_status(workspace.data_ptr(), ctypes.byref(out), _stream()),
           "qdelta_workspace_status")
    return out.value


def chunk_fwd(q, k, v, beta, alpha=None, lam=None, h0=None, chunk=64, save_for_bwd=False,
              workspace=None, o=None, hT=None, want_hT=True, logits=False, norm_qk=False):
    """Chunkwise forward.  Returns (o, hT, workspace).  All tensors live on the GPU.
    logits=True: beta, alpha, lam hold the logits of sigmoid gates (the kernels apply the sigmoid).
    norm_qk=True: q and k are un-normalised, the kernels L2-normalise them per token and head."""
    lib = load()
    s = make_shape(q, v, chunk)
    B, T, H, dk, dv, dt = s.B, s.T, s.H, s.dk, s.dv, q.dtype
    if workspace is None:
        workspace = alloc_workspace(s, save_for_bwd, q.device)
    if o is None:
        o = torch.empty((B, T, H, dv), dtype=dt, device=q.device)
    if hT is None and want_hT:
        hT = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q.device)
    rc = lib.qdelta_chunk_fwd(
        ctypes.byref(s), _ptr(q, dt, (B, T, H, dk), "q"), _ptr(k, dt, (B, T, H, dk), "k"),
        _ptr(v, dt, (B, T, H, dv), "v"), _ptr(beta, dt, (B, T, H), "beta"),
        _ptr(alpha, dt, (B, T, H), "alpha"), _ptr(lam, dt, (B, T, H), "lam"),
        _ptr(h0, torch.float32, (B, H, dk, dv), "h0"), _ptr(o, dt, (B, T, H, dv), "o"),
        _ptr(hT, torch.float32, (B, H, dk, dv), "hT"),
        workspace.data_ptr(), workspace.numel(),
        (QD_FWD_SAVE_FOR_BWD if save_for_bwd else 0) | (QD_COEF_LOGITS if logits else 0) | (QD_NORM_QK if norm_qk else 0),
        _stream())
    _check(rc, "qdelta_chunk_fwd")
    return o, hT, workspace


def chunk_fwd_static(q, k, v, beta, alpha, lam, h0, o, hT=None, status=None, chunk=64):
    """Forward on the library's built-in scratch array: no workspace, nothing allocated.

    Every output is the caller's: `o` (required), `hT` (optional fp32 final state) and `status`
    (optional int32/uint32 tensor of one element on the GPU that receives the device status word).
    """
    lib = load()
    s = make_shape(q, v, chunk)
    B, T, H, dk, dv, dt = s.B, s.T, s.H, s.dk, s.dv, q.dtype
    if o is None:
        raise QdeltaError("chunk_fwd_static: the output tensor must be supplied (this call allocates nothing)")
    sp = None
    if status is not None:
        if status.numel() != 1 or status.element_size() != 4 or not status.is_cuda:
            raise QdeltaError("chunk_fwd_static: status must be one 32-bit word on the GPU")
        sp = status.data_ptr()
    rc = lib.qdelta_chunk_fwd_static(
        ctypes.byref(s), _ptr(q, dt, (B, T, H, dk), "q"), _ptr(k, dt, (B, T, H, dk), "k"),
        _ptr(v, dt, (B, T, H, dv), "v"), _ptr(beta, dt, (B, T, H), "beta"),
        _ptr(alpha, dt, (B, T, H), "alpha"), _ptr(lam, dt, (B, T, H), "lam"),
        _ptr(h0, torch.float32, (B, H, dk, dv), "h0"), _ptr(o, dt, (B, T, H, dv), "o"),
        _ptr(hT, torch.float32, (B, H, dk, dv), "hT"), sp, _stream())
    _check(rc, "qdelta_chunk_fwd_static")
    return o, hT


def chunk_bwd(q, k, v, beta, alpha, lam, h0, dO, dhT=None, chunk=64, workspace=None,
              reuse_fwd=False, out=None, want_dh0=True, logits=False, norm_qk=False):
    """Chunkwise backward.  Returns dict(dq, dk, dv, dbeta, dalpha, dlam, dh0) of GPU tensors.
    logits=True: beta, alpha, lam are logits and dbeta, dalpha, dlam are gradients with respect to them.
    norm_qk=True: q, k are un-normalised and dq, dk are gradients with respect to them."""
    lib = load()
    s = make_shape(q, v, chunk)
    B, T, H, dk, dv, dt = s.B, s.T, s.H, s.dk, s.dv, q.dtype
    dev = q.device
    if workspace is None:
        if reuse_fwd:
            raise QdeltaError("reuse_fwd needs the workspace of the forward call")
        workspace = alloc_workspace(s, True, dev)
    g = out if out is not None else {}
    f32 = torch.float32
    g.setdefault("dq", torch.empty((B, T, H, dk), dtype=dt, device=dev))
    g.setdefault("dk", torch.empty((B, T, H, dk), dtype=dt, device=dev))
    g.setdefault("dv", torch.empty((B, T, H, dv), dtype=dt, device=dev))
    g.setdefault("dbeta", torch.empty((B, T, H), dtype=f32, device=dev))
    g.setdefault("dalpha", torch.empty((B, T, H), dtype=f32, device=dev) if alpha is not None else None)
    g.setdefault("dlam", torch.empty((B, T, H), dtype=f32, device=dev) if lam is not None else None)
    g.setdefault("dh0", torch.empty((B, H, dk, dv), dtype=f32, device=dev) if want_dh0 else None)
    rc = lib.qdelta_chunk_bwd(
        ctypes.byref(s), _ptr(q, dt, (B, T, H, dk), "q"), _ptr(k, dt, (B, T, H, dk), "k"),
        _ptr(v, dt, (B, T, H, dv), "v"), _ptr(beta, dt, (B, T, H), "beta"),
        _ptr(alpha, dt, (B, T, H), "alpha"), _ptr(lam, dt, (B, T, H), "lam"),
        _ptr(h0, f32, (B, H, dk, dv), "h0"), _ptr(dO, dt, (B, T, H, dv), "dO"),
        _ptr(dhT, f32, (B, H, dk, dv), "dhT"),
        _ptr(g["dq"], dt, (B, T, H, dk), "dq"), _ptr(g["dk"], dt, (B, T, H, dk), "dk"),
        _ptr(g["dv"], dt, (B, T, H, dv), "dv"), _ptr(g["dbeta"], f32, (B, T, H), "dbeta"),
        _ptr(g["dalpha"], f32, (B, T, H), "dalpha"), _ptr(g["dlam"], f32, (B, T, H), "dlam"),
        _ptr(g["dh0"], f32, (B, H, dk, dv), "dh0"),
        workspace.data_ptr(), workspace.numel(),
        (QD_BWD_REUSE_FWD if reuse_fwd else 0) | (QD_COEF_LOGITS if logits else 0) | (QD_NORM_QK if norm_qk else 0),
        _stream())
    _check(rc, "qdelta_chunk_bwd")
    return g


def recurrent_step(q, k, v, beta, alpha, lam, state, o=None):
    """One decode step; `state` [B,H,dk,dv] fp32 is updated in place.  Returns o [B,H,dv]."""
    lib = load()
    B, H, dk = q.shape
    dv = v.shape[-1]
    dt = q.dtype
    if o is None:
        o = torch.empty((B, H, dv), dtype=dt, device=q.device)
    rc = lib.qdelta_recurrent_step(
        B, H, dk, dv, _dtype_code(q), _ptr(q, dt, (B, H, dk), "q"), _ptr(k, dt, (B, H, dk), "k"),
        _ptr(v, dt, (B, H, dv), "v"), _ptr(beta, dt, (B, H), "beta"), _ptr(alpha, dt, (B, H), "alpha"),
        _ptr(lam, dt, (B, H), "lam"), _ptr(state, torch.float32, (B, H, dk, dv), "state"),
        _ptr(o, dt, (B, H, dv), "o"), _stream())
    _check(rc, "qdelta_recurrent_step")
    return o


def recurrent_steps(q, k, v, beta, alpha, lam, state, o=None, logits=False, norm_qk=False):
    """S decode tokens per call: q,k [B,S,H,dk], v [B,S,H,dv], coefficients [B,S,H]; `state` [B,H,dk,dv] fp32 is
    updated in place to the state after the last token.  Returns o [B,S,H,dv].  A bf16 `state` selects the
    reduced-precision state option (QD_STATE_BF16)."""
    lib = load()
    B, S, H, dk = q.shape
    dv = v.shape[-1]
    dt = q.dtype
    if state.dtype not in (torch.float32, torch.bfloat16):
        raise QdeltaError("state must be fp32, or bf16 for the reduced-precision state option")
    state_bf16 = state.dtype == torch.bfloat16
    if o is None:
        o = torch.empty((B, S, H, dv), dtype=dt, device=q.device)
    rc = lib.qdelta_recurrent_steps(
        B, S, H, dk, dv, _dtype_code(q), _ptr(q, dt, (B, S, H, dk), "q"), _ptr(k, dt, (B, S, H, dk), "k"),
        _ptr(v, dt, (B, S, H, dv), "v"), _ptr(beta, dt, (B, S, H), "beta"), _ptr(alpha, dt, (B, S, H), "alpha"),
        _ptr(lam, dt, (B, S, H), "lam"), _ptr(state, None, (B, H, dk, dv), "state"),
        _ptr(o, dt, (B, S, H, dv), "o"),
        (QD_COEF_LOGITS if logits else 0) | (QD_NORM_QK if norm_qk else 0) | (QD_STATE_BF16 if state_bf16 else 0), _stream())
    _check(rc, "qdelta_recurrent_steps")
    return o
