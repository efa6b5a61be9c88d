"""ctypes front-end of the fp64 recurrence oracle (``qdelta_oracle.c``).

TEST INFRASTRUCTURE ONLY (see the package docstring).  Every array is converted
to contiguous float64 before the call; layouts are token-major:
q,k [B,T,H,dk]; v,o,dO [B,T,H,dv]; beta,alpha,lam [B,T,H]; states [B,H,dk,dv].
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.qd_oracle_fwd.restype = ctypes.c_int
        lib.qd_oracle_fwd.argtypes = [ctypes.c_int] * 5 + [dp] * 9
        lib.qd_oracle_bwd.restype = ctypes.c_int
        lib.qd_oracle_bwd.argtypes = [ctypes.c_int] * 6 + [dp] * 16
        lib.qd_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _c(a, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _p(a):
    if a is None:
        return ctypes.POINTER(ctypes.c_double)()
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def max_threads() -> int:
    return int(_load().qd_oracle_max_threads())


def forward(q, k, v, beta, alpha=None, lam=None, h0=None):
    """Token-by-token Q-Delta recurrence (Section 3.3.1).  Returns (o, hT)."""
    lib = _load()
    q = _c(q)
    B, T, H, dk = q.shape
    dv = np.shape(v)[-1]
    k = _c(k, (B, T, H, dk)); v = _c(v, (B, T, H, dv))
    beta = _c(beta, (B, T, H)); alpha = _c(alpha, (B, T, H)); lam = _c(lam, (B, T, H))
    h0 = _c(h0, (B, H, dk, dv))
    o = np.empty((B, T, H, dv), np.float64)
    hT = np.empty((B, H, dk, dv), np.float64)
    rc = lib.qd_oracle_fwd(B, T, H, dk, dv, _p(q), _p(k), _p(v), _p(beta), _p(alpha),
                           _p(lam), _p(h0), _p(o), _p(hT))
    if rc != 0:
        raise RuntimeError("qd_oracle_fwd failed: %d" % rc)
    return o, hT


def backward(q, k, v, beta, alpha, lam, h0, dO, dhT=None, ckpt=64):
    """Reverse pass of the recurrence for L = <o,dO> + <hT,dhT>.

    Returns dict(dq, dk, dv, dbeta, dalpha, dlam, dh0); dalpha is the derivative
    with respect to alpha itself.  alpha=None means alpha==1, lam=None means 0
    (their gradients are still returned)."""
    lib = _load()
    q = _c(q)
    B, T, H, dk = q.shape
    dv = np.shape(v)[-1]
    k = _c(k, (B, T, H, dk)); v = _c(v, (B, T, H, dv))
    beta = _c(beta, (B, T, H)); alpha = _c(alpha, (B, T, H)); lam = _c(lam, (B, T, H))
    h0 = _c(h0, (B, H, dk, dv)); dO = _c(dO, (B, T, H, dv)); dhT = _c(dhT, (B, H, dk, dv))
    out = dict(dq=np.empty((B, T, H, dk)), dk=np.empty((B, T, H, dk)),
               dv=np.empty((B, T, H, dv)), dbeta=np.empty((B, T, H)),
               dalpha=np.empty((B, T, H)), dlam=np.empty((B, T, H)),
               dh0=np.empty((B, H, dk, dv)))
    rc = lib.qd_oracle_bwd(B, T, H, dk, dv, int(ckpt), _p(q), _p(k), _p(v), _p(beta),
                           _p(alpha), _p(lam), _p(h0), _p(dO), _p(dhT),
                           _p(out["dq"]), _p(out["dk"]), _p(out["dv"]), _p(out["dbeta"]),
                           _p(out["dalpha"]), _p(out["dlam"]), _p(out["dh0"]))
    if rc != 0:
        raise RuntimeError("qd_oracle_bwd failed: %d" % rc)
    return out


def decode(state, q, k, v, beta, alpha=None, lam=None):
    """`steps` single-token updates of [Bn,H,dk,dv] states.

    q,k [steps,Bn,H,dk], v [steps,Bn,H,dv], coefficients [steps,Bn,H].
    Returns (o [steps,Bn,H,dv], final state).  It is the forward recurrence
    with time as the leading axis."""
    tr = lambda a: None if a is None else np.moveaxis(np.asarray(a, np.float64), 0, 1)
    o, hT = forward(tr(q), tr(k), tr(v), tr(beta), tr(alpha), tr(lam), state)
    return np.moveaxis(o, 1, 0), hT


def _sigmoid(z):
    """sigma(z) in fp64 without overflow for large |z|."""
    z = np.asarray(z, np.float64)
    e = np.exp(-np.abs(z))
    return np.where(z >= 0, 1.0 / (1.0 + e), e / (1.0 + e))


def gates_from_logits(zbeta, zalpha=None, zlam=None):
    """The coefficients as sigmoid gates of pre-activation logits (Appendix B writes lambda this way; beta and alpha
    are gates in (0,1) as well).  An absent alpha / lambda stays absent (alpha == 1, lambda == 0)."""
    g = lambda z: None if z is None else _sigmoid(z)
    return _sigmoid(zbeta), g(zalpha), g(zlam)


def forward_logits(q, k, v, zbeta, zalpha=None, zlam=None, h0=None):
    """forward() with beta, alpha, lambda given as logits."""
    beta, alpha, lam = gates_from_logits(zbeta, zalpha, zlam)
    return forward(q, k, v, beta, alpha, lam, h0)


def backward_logits(q, k, v, zbeta, zalpha, zlam, h0, dO, dhT=None, ckpt=64):
    """backward() with beta, alpha, lambda given as logits: dbeta, dalpha, dlam are the derivatives with respect to the
    logits, by the chain rule d sigma(z)/dz = sigma(z)(1 - sigma(z)).  Gradients of absent logits are returned as None."""
    beta, alpha, lam = gates_from_logits(zbeta, zalpha, zlam)
    g = backward(q, k, v, beta, alpha, lam, h0, dO, dhT, ckpt)
    g["dbeta"] = g["dbeta"] * beta * (1.0 - beta)
    g["dalpha"] = None if alpha is None else g["dalpha"] * alpha * (1.0 - alpha)
    g["dlam"] = None if lam is None else g["dlam"] * lam * (1.0 - lam)
    return g


NORM_EPS = 1e-6


def l2_normalize(x):
    """x / sqrt(|x|^2 + NORM_EPS) along the last axis (per token and head), fp64.  The text gives no formula for the
    normalisation of q and k; this is the usual L2 normalisation with a small constant under the root."""
    x = np.asarray(x, np.float64)
    return x / np.sqrt(np.sum(x * x, axis=-1, keepdims=True) + NORM_EPS)


def l2_normalize_backward(x, dxhat):
    """Gradient through l2_normalize: with r = 1/sqrt(|x|^2 + eps) and x^ = r x,  dx = r (dx^ - x^ <x^, dx^>)."""
    x = np.asarray(x, np.float64)
    r = 1.0 / np.sqrt(np.sum(x * x, axis=-1, keepdims=True) + NORM_EPS)
    xh = r * x
    return r * (dxhat - xh * np.sum(xh * dxhat, axis=-1, keepdims=True))


def forward_fused(q, k, v, beta, alpha=None, lam=None, h0=None, logits=False, norm_qk=False):
    """forward() behind the optional pre-processing stages: L2 normalisation of q and k, gates from logits."""
    if norm_qk:
        q, k = l2_normalize(q), l2_normalize(k)
    if logits:
        beta, alpha, lam = gates_from_logits(beta, alpha, lam)
    return forward(q, k, v, beta, alpha, lam, h0)


def backward_fused(q, k, v, beta, alpha, lam, h0, dO, dhT=None, ckpt=64, logits=False, norm_qk=False):
    """backward() behind the same stages: gradients with respect to what the caller passed in."""
    qn, kn = (l2_normalize(q), l2_normalize(k)) if norm_qk else (q, k)
    if logits:
        g = backward_logits(qn, kn, v, beta, alpha, lam, h0, dO, dhT, ckpt)
    else:
        g = backward(qn, kn, v, beta, alpha, lam, h0, dO, dhT, ckpt)
    if norm_qk:
        g["dq"] = l2_normalize_backward(q, g["dq"])
        g["dk"] = l2_normalize_backward(k, g["dk"])
    return g
