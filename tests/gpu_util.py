"""Helpers of the GPU parity tests: move seeded inputs to the device, compare with the oracle."""
import numpy as np
import torch

from oracle import recurrence as orc

TOL = {"f32": 1e-4, "bf16": 2e-2}     # per tensor: max|gpu - ref| / max|ref|  (the contract's bar)
# Two stricter companions of that bar, asserted wherever the oracle covers whole sequences:
#   rms      sqrt(mean (gpu - ref)^2) / sqrt(mean ref^2) over the tensor;
#   per_seq  max|gpu - ref| / max|ref| taken separately over every (batch, head) sequence, worst sequence reported
#            (one large entry elsewhere in the tensor cannot hide a bad sequence).
TOL_RMS = {"f32": 5e-5, "bf16": 1e-2}
TOL_SEQ = {"f32": 1e-4, "bf16": 2e-2}     # the contract's bar, but met by every sequence on its own
LOG = []                               # (label, tensor name, max, rms, per_seq) of every comparison, dumped by conftest
TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


def to_dev(a, dtype):
    if a is None:
        return None
    return torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dtype)


def dev_inputs(d, dtype):
    """numpy input dict -> torch CUDA tensors (q,k,v,coefficients,dO in `dtype`; states fp32)."""
    t = TDT[dtype]
    out = {n: to_dev(d.get(n), t) for n in ("q", "k", "v", "beta", "alpha", "lam", "dO")}
    out["h0"] = to_dev(d.get("h0"), torch.float32)
    out["dhT"] = to_dev(d.get("dhT"), torch.float32)
    return out


def rel_err(gpu, ref):
    gpu = gpu.detach().to(torch.float64).cpu().numpy()
    ref = np.asarray(ref, np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), "non-finite values in GPU result"
    den = np.max(np.abs(ref))
    return float(np.max(np.abs(gpu - ref)) / (den if den > 0 else 1.0))


def errors(gpu, ref, state=False):
    """(max-normalised, rms-relative, worst per-sequence) error of a result against the oracle.
    Token tensors are [B,T,H,...] (sequence = fixed b and h), states are [B,H,dk,dv]."""
    gpu = gpu.detach().to(torch.float64).cpu().numpy()
    ref = np.asarray(ref, np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), "non-finite values in GPU result"
    diff = np.abs(gpu - ref)
    den = np.max(np.abs(ref))
    emax = float(np.max(diff) / (den if den > 0 else 1.0))
    r2 = float(np.sqrt(np.mean(ref * ref)))
    erms = float(np.sqrt(np.mean(diff * diff)) / (r2 if r2 > 0 else 1.0))
    if state:
        ax = tuple(range(2, ref.ndim))
        dseq, rseq = diff.max(axis=ax), np.abs(ref).max(axis=ax)
    else:
        ax = (1,) + tuple(range(3, ref.ndim))
        dseq, rseq = diff.max(axis=ax), np.abs(ref).max(axis=ax)
    eseq = float(np.max(dseq / np.where(rseq > 0, rseq, 1.0)))
    return emax, erms, eseq


def check(label, name, gpu, ref, dtype, state=False):
    """Assert all three bars for one tensor and log the figures."""
    emax, erms, eseq = errors(gpu, ref, state)
    LOG.append((label, name, emax, erms, eseq))
    assert emax <= TOL[dtype] and erms <= TOL_RMS[dtype] and eseq <= TOL_SEQ[dtype], (label, name, emax, erms, eseq)
    return emax


def all_finite(*tensors):
    return all(bool(torch.isfinite(t.float()).all().item()) for t in tensors if t is not None)


class Guarded:
    """A CUDA tensor inside a larger allocation with a band of a fixed byte pattern on either side.
    intact() tells whether a kernel wrote outside the tensor (compute-sanitizer is not available here)."""
    BAND = 4096
    PATTERN = 0xA5

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = n
        pad = (-n) % 16
        self.raw = torch.full((self.BAND + n + pad + self.BAND,), self.PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.BAND:self.BAND + n].view(dtype).view(*shape)
        if fill is not None:
            self.t.copy_(fill)

    def intact(self):
        lo = self.raw[:self.BAND]
        hi = self.raw[self.BAND + self.nbytes:]
        return bool((lo == self.PATTERN).all().item()) and bool((hi == self.PATTERN).all().item())


def pick_sequences(d, pairs):
    """Sub-problem made of the (b,h) sequences in `pairs`, as B'=len(pairs), H'=1."""
    out = {}
    for n, a in d.items():
        if a is None:
            out[n] = None
        elif n in ("h0", "dhT"):
            out[n] = np.stack([a[b, h][None] for b, h in pairs])
        else:
            out[n] = np.stack([a[b, :, h][:, None] for b, h in pairs])
    return out


def pick_result(t, pairs, state=False):
    """Matching slice of a GPU result tensor."""
    if state:
        return torch.stack([t[b, h][None] for b, h in pairs])
    return torch.stack([t[b, :, h][:, None] for b, h in pairs])


def oracle_fwd(d):
    return orc.forward(d["q"], d["k"], d["v"], d["beta"], d.get("alpha"), d.get("lam"), d.get("h0"))


def oracle_bwd(d):
    return orc.backward(d["q"], d["k"], d["v"], d["beta"], d.get("alpha"), d.get("lam"), d.get("h0"),
                        d["dO"], d.get("dhT"))
