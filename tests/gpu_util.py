"""Helpers of the GPU parity tests: move seeded inputs to the device, compare with the oracle."""
import numpy as np
import torch

from oracle import recurrence as orc

TOL = {"f32": 1e-4, "bf16": 2e-2}     # per tensor: max|gpu - ref| / max|ref|
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
