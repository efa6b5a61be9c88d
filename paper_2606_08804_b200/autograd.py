"""`torch.autograd` front-end of the chunkwise kernels: marshalling only.

    o, hT = qdelta_chunk(q, k, v, beta, alpha, lam, h0, logits=False, norm_qk=False)

q, k [B,T,H,dk], v [B,T,H,dv], beta/alpha/lam [B,T,H] (alpha, lam, h0 may be None), all CUDA tensors; returns the
outputs o [B,T,H,dv] and the final state hT [B,H,dk,dv] (fp32), both differentiable.  The forward runs
`qdelta_chunk_fwd` saving what the backward needs in a workspace that the autograd node keeps; the backward runs
`qdelta_chunk_bwd` on that workspace.  Every number is computed by the library's CUDA kernels.
"""
import torch

from . import binding as qd


class _QDeltaChunk(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, beta, alpha, lam, h0, logits, norm_qk):
        c = lambda t: None if t is None else t.contiguous()
        q, k, v, beta, alpha, lam, h0 = (c(t) for t in (q, k, v, beta, alpha, lam, h0))
        need_grad = any(t is not None and t.requires_grad for t in (q, k, v, beta, alpha, lam, h0))
        o, hT, ws = qd.chunk_fwd(q, k, v, beta, alpha, lam, h0, save_for_bwd=need_grad, logits=logits, norm_qk=norm_qk)
        ctx.save_for_backward(q, k, v, beta, alpha, lam, h0)
        ctx.ws, ctx.logits, ctx.norm_qk = (ws if need_grad else None), logits, norm_qk
        return o, hT

    @staticmethod
    def backward(ctx, dO, dhT):
        q, k, v, beta, alpha, lam, h0 = ctx.saved_tensors
        dO = torch.zeros_like(v) if dO is None else dO.contiguous()
        dhT = None if dhT is None else dhT.contiguous().float()
        g = qd.chunk_bwd(q, k, v, beta, alpha, lam, h0, dO, dhT, workspace=ctx.ws, reuse_fwd=ctx.ws is not None,
                         want_dh0=h0 is not None, logits=ctx.logits, norm_qk=ctx.norm_qk)
        coef = lambda name, ref: None if ref is None else g[name].to(ref.dtype)
        return (g["dq"], g["dk"], g["dv"], coef("dbeta", beta), coef("dalpha", alpha), coef("dlam", lam),
                g["dh0"] if h0 is not None else None, None, None)


def qdelta_chunk(q, k, v, beta, alpha=None, lam=None, h0=None, logits=False, norm_qk=False):
    """Differentiable chunkwise Q-Delta: returns (o, hT)."""
    return _QDeltaChunk.apply(q, k, v, beta, alpha, lam, h0, bool(logits), bool(norm_qk))
